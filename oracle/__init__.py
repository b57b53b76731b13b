"""ctypes front end of the CPU oracle (``srq_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the bench's CPU
baseline leg import this; the product package never does, and this module
never imports the product package.  The arithmetic lives in the C file; this
module builds it with gcc and marshals numpy arrays.  One exception, stated
where it occurs: qlinear_fwd_fp_act forms its binary64 product with numpy's
matmul (a library routine used as one step) around the C quantizer.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "srq_oracle.c")
_LIB = os.path.join(_HERE, "libsrq_oracle.so")

PER_TENSOR, PER_ROW = 0, 1
SR, RTN, SR8 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _QSpec(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int32), ("scale_mode", ctypes.c_int32),
                ("round_mode", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("seed", ctypes.c_uint64), ("tensor_id", ctypes.c_uint64),
                ("index_offset", ctypes.c_uint64)]


@dataclass
class QSpec:
    """One quantization point: the (Delta rule, eps) pair of one operand."""
    bits: int = 8
    scale_mode: int = PER_TENSOR
    round_mode: int = SR
    seed: int = 0
    tensor_id: int = 0
    index_offset: int = 0

    def c(self) -> _QSpec:
        return _QSpec(self.bits, self.scale_mode, self.round_mode, 0, self.seed, self.tensor_id,
                      self.index_offset)


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        L = _lib
        u32p = ctypes.POINTER(ctypes.c_uint32)
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_philox4x32_10.restype = None
        L.orc_threshold_u24.argtypes = [ctypes.c_uint64] * 3
        L.orc_threshold_u24.restype = ctypes.c_uint32
        L.orc_threshold_sr8.argtypes = [ctypes.c_uint64] * 3
        L.orc_threshold_sr8.restype = ctypes.c_uint32
        L.orc_scale_from_absmax.argtypes = [ctypes.c_float, ctypes.c_int,
                                            ctypes.POINTER(ctypes.c_float),
                                            ctypes.POINTER(ctypes.c_float)]
        L.orc_scale_from_absmax.restype = None
        L.orc_quantize_scalar.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_uint32]
        L.orc_quantize_scalar.restype = ctypes.c_int
        vp = ctypes.c_void_p
        i64 = ctypes.c_int64
        L.orc_sum_sr_codes_over_all_thresholds.argtypes = [ctypes.c_float, ctypes.c_float,
                                                          ctypes.c_int]
        L.orc_sum_sr_codes_over_all_thresholds.restype = i64
        for name in ("orc_absmax_tensor", "orc_absmax_rows", "orc_absmax_cols"):
            getattr(L, name).argtypes = [vp, i64, i64, i64, vp]
            getattr(L, name).restype = None
        L.orc_sr_quantize.argtypes = [vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                                      vp, vp, vp, vp]
        L.orc_sr_quantize.restype = ctypes.c_int
        L.orc_gemm_i8_nt.argtypes = [vp, vp, i64, i64, i64, vp]
        L.orc_gemm_i8_nt.restype = i64
        L.orc_dequant.argtypes = [vp, i64, i64, vp, ctypes.c_int, vp, ctypes.c_int, vp]
        L.orc_dequant.restype = None
        qp = ctypes.POINTER(_QSpec)
        for name in ("orc_qlinear_fwd", "orc_qlinear_bwd_input", "orc_qlinear_bwd_weight"):
            getattr(L, name).argtypes = [vp, vp, i64, i64, i64, qp, qp, vp, vp, vp, vp, vp, vp]
            getattr(L, name).restype = i64
        L.orc_e4m3_decode.argtypes = [ctypes.c_uint8]
        L.orc_e4m3_decode.restype = ctypes.c_double
        L.orc_quantize_e4m3_scalar.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_uint32]
        L.orc_quantize_e4m3_scalar.restype = ctypes.c_uint8
        L.orc_scale_e4m3.argtypes = [ctypes.c_float, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]
        L.orc_scale_e4m3.restype = None
        L.orc_sr_quantize_e4m3.argtypes = [vp, i64, i64, i64, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, vp, vp, vp, vp]
        L.orc_sr_quantize_e4m3.restype = ctypes.c_int
        L.orc_e4m_max.argtypes = [ctypes.c_int]
        L.orc_e4m_max.restype = ctypes.c_double
        L.orc_quantize_e4m_scalar.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_uint32]
        L.orc_quantize_e4m_scalar.restype = ctypes.c_uint8
        L.orc_scale_e4m.argtypes = [ctypes.c_float, ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]
        L.orc_scale_e4m.restype = None
        L.orc_sr_quantize_e4m.argtypes = [vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, vp, vp, vp, vp]
        L.orc_sr_quantize_e4m.restype = ctypes.c_int
        L.orc_gemm_e4m3_nt.argtypes = [vp, vp, i64, i64, i64, vp, ctypes.c_int, vp, ctypes.c_int, vp, vp]
        L.orc_gemm_e4m3_nt.restype = None
        L.orc_requantize.argtypes = [vp, i64, i64, ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_uint64,
                                     ctypes.c_uint64, ctypes.c_uint64, vp, ctypes.POINTER(ctypes.c_float)]
        L.orc_requantize.restype = None
        L.orc_accumulate.argtypes = [vp, vp, i64]
        L.orc_accumulate.restype = None
        L.orc_to_bf16.argtypes = [vp, i64, vp]
        L.orc_to_bf16.restype = None
        L.orc_num_threads.argtypes = []
        L.orc_num_threads.restype = ctypes.c_int
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32_2d(x) -> np.ndarray:
    x = np.asarray(x)
    if x.dtype != np.float32 or x.ndim != 2:
        raise TypeError("oracle takes 2-D float32 arrays (widen bfloat16 first)")
    if x.strides[1] != 4 or x.strides[0] % 4 != 0:
        x = np.ascontiguousarray(x)
    return x


def num_threads() -> int:
    return int(lib().orc_num_threads())


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (ctypes.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def threshold_u24(seed: int, tensor_id: int, i: int) -> int:
    return int(lib().orc_threshold_u24(seed, tensor_id, i))


def threshold_sr8(seed: int, tensor_id: int, i: int) -> int:
    """Threshold of element i in the 8-random-bit mode, on the 2^-24 lattice: (2 b + 1) 2^15."""
    return int(lib().orc_threshold_sr8(seed, tensor_id, i))


def scale_from_absmax(m: float, bits: int):
    d, inv = ctypes.c_float(), ctypes.c_float()
    lib().orc_scale_from_absmax(ctypes.c_float(m), bits, ctypes.byref(d), ctypes.byref(inv))
    return np.float32(d.value), np.float32(inv.value)


def quantize_scalar(x: float, inv: float, bits: int, round_mode: int, u24: int = 0) -> int:
    return int(lib().orc_quantize_scalar(ctypes.c_float(x), ctypes.c_float(inv), bits, round_mode,
                                         u24))


def sum_sr_codes_over_all_thresholds(x: float, inv: float, bits: int) -> int:
    return int(lib().orc_sum_sr_codes_over_all_thresholds(ctypes.c_float(x), ctypes.c_float(inv),
                                                         bits))


def absmax(x, mode: str) -> np.ndarray:
    x = _f32_2d(x)
    rows, cols = x.shape
    ld = x.strides[0] // 4
    n = {"tensor": 1, "rows": rows, "cols": cols}[mode]
    m = np.zeros(n, dtype=np.float32)
    getattr(lib(), "orc_absmax_" + mode)(_ptr(x), rows, cols, ld, _ptr(m))
    return m


def sr_quantize(x, q: QSpec, want_rm: bool = True, want_tr: bool = False):
    """Returns (codes_rm, scale_rm, codes_tr, scale_tr); unrequested pairs are None."""
    x = _f32_2d(x)
    rows, cols = x.shape
    ld = x.strides[0] // 4
    per_row = q.scale_mode == PER_ROW
    crm = srm = ctr = strr = None
    if want_rm:
        crm = np.zeros((rows, cols), dtype=np.int8)
        srm = np.zeros(rows if per_row else 1, dtype=np.float32)
    if want_tr:
        ctr = np.zeros((cols, rows), dtype=np.int8)
        strr = np.zeros(cols if per_row else 1, dtype=np.float32)
    rc = lib().orc_sr_quantize(_ptr(x), rows, cols, ld, q.bits, q.scale_mode, q.round_mode,
                               q.seed, q.tensor_id, q.index_offset,
                               _ptr(crm), _ptr(srm), _ptr(ctr), _ptr(strr))
    if rc != 0:
        raise ValueError("oracle: bits outside 2..8")
    return crm, srm, ctr, strr


def gemm_i8_nt(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """acc[i,j] = sum_k a[i,k] b[j,k] for int8 codes; raises if a sum leaves int32."""
    a = np.ascontiguousarray(a, dtype=np.int8)
    b = np.ascontiguousarray(b, dtype=np.int8)
    M, Kc = a.shape
    N, Kb = b.shape
    assert Kc == Kb
    acc = np.zeros((M, N), dtype=np.int32)
    ov = lib().orc_gemm_i8_nt(_ptr(a), _ptr(b), M, N, Kc, _ptr(acc))
    if ov:
        raise OverflowError(f"{ov} accumulators do not fit in int32")
    return acc


def dequant(acc: np.ndarray, s_row: np.ndarray, s_col: np.ndarray) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    s_row = np.ascontiguousarray(s_row, dtype=np.float32)
    s_col = np.ascontiguousarray(s_col, dtype=np.float32)
    M, N = acc.shape
    assert s_row.size in (1, M) and s_col.size in (1, N)
    out = np.zeros((M, N), dtype=np.float32)
    lib().orc_dequant(_ptr(acc), M, N, _ptr(s_row), int(s_row.size != 1),
                      _ptr(s_col), int(s_col.size != 1), _ptr(out))
    return out


@dataclass
class LinearResult:
    out: np.ndarray
    acc: np.ndarray
    codes_a: np.ndarray
    scale_a: np.ndarray
    codes_b: np.ndarray
    scale_b: np.ndarray


def _qlinear(fn, X0, X1, T, N, K, q0: QSpec, q1: QSpec, shape0, shape1, out_shape):
    X0 = np.ascontiguousarray(X0, dtype=np.float32)
    X1 = np.ascontiguousarray(X1, dtype=np.float32)
    c0 = np.zeros(shape0, dtype=np.int8)
    c1 = np.zeros(shape1, dtype=np.int8)
    s0 = np.zeros(shape0[0] if q0.scale_mode == PER_ROW else 1, dtype=np.float32)
    s1 = np.zeros(shape1[0] if q1.scale_mode == PER_ROW else 1, dtype=np.float32)
    acc = np.zeros(out_shape, dtype=np.int32)
    out = np.zeros(out_shape, dtype=np.float32)
    c_q0, c_q1 = q0.c(), q1.c()
    ov = fn(_ptr(X0), _ptr(X1), T, N, K, ctypes.byref(c_q0), ctypes.byref(c_q1),
            _ptr(c0), _ptr(s0), _ptr(c1), _ptr(s1), _ptr(acc), _ptr(out))
    if ov:
        raise OverflowError(f"{ov} accumulators do not fit in int32")
    return LinearResult(out, acc, c0, s0, c1, s1)


def qlinear_fwd(A, W, qa: QSpec, qw: QSpec) -> LinearResult:
    """Alg. 1: Y[T,N] = Q(A[T,K]) Q(W[N,K])^T."""
    T, K = A.shape
    N, K2 = W.shape
    assert K == K2
    return _qlinear(lib().orc_qlinear_fwd, A, W, T, N, K, qa, qw, (T, K), (N, K), (T, N))


def qlinear_bwd_input(dY, W, qdy: QSpec, qw: QSpec) -> LinearResult:
    """Alg. 2: dA[T,K] = Q(dY[T,N]) Q(W[N,K]); codes_b is the [K,N] layout of Q(W)."""
    T, N = dY.shape
    N2, K = W.shape
    assert N == N2
    return _qlinear(lib().orc_qlinear_bwd_input, dY, W, T, N, K, qdy, qw, (T, N), (K, N), (T, K))


def qlinear_bwd_weight(dY, A, qdy: QSpec, qa: QSpec) -> LinearResult:
    """Alg. 2: dW[N,K] = Q(dY[T,N])^T Q(A[T,K]); both code sets are transposed layouts."""
    T, N = dY.shape
    T2, K = A.shape
    assert T == T2
    return _qlinear(lib().orc_qlinear_bwd_weight, dY, A, T, N, K, qdy, qa, (N, T), (K, T), (N, K))


# ---------------------------------------------------------------------------------------------
# E4M3 grid
# ---------------------------------------------------------------------------------------------
def e4m3_decode(codes) -> np.ndarray:
    """Values (binary64) of E4M3 code bytes."""
    table = np.array([lib().orc_e4m3_decode(i) for i in range(256)], dtype=np.float64)
    return table[np.asarray(codes, dtype=np.uint8)]


def scale_e4m3(m: float):
    d, inv = ctypes.c_float(), ctypes.c_float()
    lib().orc_scale_e4m3(ctypes.c_float(m), ctypes.byref(d), ctypes.byref(inv))
    return np.float32(d.value), np.float32(inv.value)


def quantize_e4m3_scalar(x: float, inv: float, round_mode: int, u24: int = 0) -> int:
    return int(lib().orc_quantize_e4m3_scalar(ctypes.c_float(x), ctypes.c_float(inv), round_mode, u24))


def e4m_max(mant: int) -> float:
    """Largest value of the E4Mk grid (k = mant mantissa bits)."""
    return float(lib().orc_e4m_max(mant))


def scale_e4m(m: float, mant: int):
    d, inv = ctypes.c_float(), ctypes.c_float()
    lib().orc_scale_e4m(ctypes.c_float(m), mant, ctypes.byref(d), ctypes.byref(inv))
    return np.float32(d.value), np.float32(inv.value)


def quantize_e4m_scalar(x: float, inv: float, mant: int, round_mode: int, u24: int = 0) -> int:
    return int(lib().orc_quantize_e4m_scalar(ctypes.c_float(x), ctypes.c_float(inv), mant, round_mode, u24))


def sr_quantize_e4m3(x, q: QSpec, want_rm: bool = True, want_tr: bool = False):
    """Def. 1-3 on the E4Mk grid, k = q.bits - 5 mantissa bits (8: E4M3, 7: E4M2, 6: E4M1, 5: E4M0);
    codes are E4M3 bytes; returns (codes_rm, scale_rm, codes_tr, scale_tr)."""
    mant = q.bits - 5
    assert 0 <= mant <= 3
    x = _f32_2d(x)
    rows, cols = x.shape
    ld = x.strides[0] // 4
    per_row = q.scale_mode == PER_ROW
    crm = srm = ctr = strr = None
    if want_rm:
        crm = np.zeros((rows, cols), dtype=np.uint8)
        srm = np.zeros(rows if per_row else 1, dtype=np.float32)
    if want_tr:
        ctr = np.zeros((cols, rows), dtype=np.uint8)
        strr = np.zeros(cols if per_row else 1, dtype=np.float32)
    lib().orc_sr_quantize_e4m(_ptr(x), rows, cols, ld, mant, q.scale_mode, q.round_mode, q.seed, q.tensor_id,
                              q.index_offset, _ptr(crm), _ptr(srm), _ptr(ctr), _ptr(strr))
    return crm, srm, ctr, strr


def gemm_e4m3_nt(a, b, s_row, s_col):
    """(acc, out) in binary64: acc[i,j] = sum_k val(a[i,k]) val(b[j,k]), out = acc * (s_row x s_col)."""
    a = np.ascontiguousarray(a, dtype=np.uint8)
    b = np.ascontiguousarray(b, dtype=np.uint8)
    s_row = np.ascontiguousarray(s_row, dtype=np.float32)
    s_col = np.ascontiguousarray(s_col, dtype=np.float32)
    M, Kc = a.shape
    N, Kb = b.shape
    assert Kc == Kb and s_row.size in (1, M) and s_col.size in (1, N)
    acc = np.zeros((M, N), dtype=np.float64)
    out = np.zeros((M, N), dtype=np.float64)
    lib().orc_gemm_e4m3_nt(_ptr(a), _ptr(b), M, N, Kc, _ptr(s_row), int(s_row.size != 1),
                           _ptr(s_col), int(s_col.size != 1), _ptr(acc), _ptr(out))
    return acc, out


def _qlinear_e4m3(X0, X1, q0, q1, tr0, tr1):
    c0 = sr_quantize_e4m3(X0, q0, not tr0, tr0)
    c1 = sr_quantize_e4m3(X1, q1, not tr1, tr1)
    ca, sa = (c0[2], c0[3]) if tr0 else (c0[0], c0[1])
    cb, sb = (c1[2], c1[3]) if tr1 else (c1[0], c1[1])
    acc, out = gemm_e4m3_nt(ca, cb, sa, sb)
    return LinearResult(out, acc, ca, sa, cb, sb)


def qlinear_fwd_e4m3(A, W, qa: QSpec, qw: QSpec) -> LinearResult:
    """Alg. 1 on the E4M3 grid: Y = Q(A) Q(W)^T (out and acc in binary64)."""
    return _qlinear_e4m3(A, W, qa, qw, False, False)


def qlinear_bwd_input_e4m3(dY, W, qdy: QSpec, qw: QSpec) -> LinearResult:
    return _qlinear_e4m3(dY, W, qdy, qw, False, True)


def qlinear_bwd_weight_e4m3(dY, A, qdy: QSpec, qa: QSpec) -> LinearResult:
    return _qlinear_e4m3(dY, A, qdy, qa, True, True)


def qlinear_fwd_fp_act(A, W, qw: QSpec) -> LinearResult:
    """Forward pass of the paper's mixed-precision SGD for the quantization-aware objective
    (Sec. 3.3: D_A^fwd = 0, only W is quantized): Y = A Q(W)^T with A as given, in binary64.
    acc holds A codes(W)^T, out = acc * D_W."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    cw, sw, _, _ = sr_quantize(W, qw, True, False)
    acc = A.astype(np.float64) @ cw.astype(np.float64).T          # library matmul as one step
    out = acc * np.broadcast_to(sw.astype(np.float64), (cw.shape[0],))[None, :]
    return LinearResult(out, acc, None, None, cw, sw)


def requantize(out, step: float, q: QSpec):
    """(codes int8 [M, N], max |out|) of a product's output quantized with a caller-supplied step."""
    out = np.ascontiguousarray(out, dtype=np.float32)
    M, N = out.shape
    codes = np.zeros((M, N), dtype=np.int8)
    m = ctypes.c_float()
    lib().orc_requantize(_ptr(out), M, N, ctypes.c_float(step), q.bits, q.round_mode, q.seed, q.tensor_id,
                         q.index_offset, _ptr(codes), ctypes.byref(m))
    return codes, np.float32(m.value)


def accumulate(dst, src) -> np.ndarray:
    """dst + src in binary32 (one addition per element), as a new array."""
    d = np.array(dst, dtype=np.float32, order="C", copy=True)
    s = np.ascontiguousarray(src, dtype=np.float32)
    assert d.shape == s.shape
    lib().orc_accumulate(_ptr(d), _ptr(s), d.size)
    return d


def to_bf16(x) -> np.ndarray:
    """Bit patterns (uint16) of the bfloat16 numbers nearest to the binary32 values, ties to even."""
    v = np.ascontiguousarray(x, dtype=np.float32)
    out = np.zeros(v.shape, dtype=np.uint16)
    lib().orc_to_bf16(_ptr(v), v.size, _ptr(out))
    return out
