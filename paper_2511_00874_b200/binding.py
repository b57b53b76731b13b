"""Thin ctypes binding of libsrq.so: argument marshalling only.

Every function has the name and argument order of the C entry point it calls (see
``include/srq.h``); tensors are torch CUDA tensors used purely as device memory, and the
current torch stream is passed as the CUDA stream.  There is no fallback: if the shared
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsrq.so")

# enums of srq.h
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_ACC_OVERFLOW, ERR_CUDA, ERR_NONFINITE, \
    ERR_TIMEOUT = range(8)
F32, BF16 = 0, 1
PER_TENSOR, PER_ROW = 0, 1
SR, RTN, SR8 = 0, 1, 2
GRID_INT, GRID_E4M3, GRID_NONE = 0, 1, 2

EXPORTS = ["srq_quantize_workspace_bytes", "srq_gemm_workspace_bytes", "srq_workspace_bytes",
           "sr_quantize", "sr_quantize_static", "srq_absmax", "srq_absmax_cols", "srq_gemm_i8", "srq_gemm_e4m3", "qlinear_fwd", "qlinear_bwd_input", "qlinear_bwd_weight", "qlinear_bwd",
           "srq_gemm_i8_ex", "qlinear_fwd_ex", "qlinear_bwd_ex", "srq_dequant_i32",
           "srq_poll_status", "srq_status_string", "srq_launch_count", "srq_selftest_bounded_wait", "srq_selftest_mma_rate", "srq_set_product_timer", "srq_plan_splits"]


class SrqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _QSpec(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int32), ("scale", ctypes.c_int32), ("round", ctypes.c_int32),
                ("format", ctypes.c_int32), ("seed", ctypes.c_uint64),
                ("tensor_id", ctypes.c_uint64), ("index_offset", ctypes.c_uint64),
                ("absmax", ctypes.c_void_p)]


class _DebugOut(ctypes.Structure):
    _fields_ = [("codes_a", ctypes.c_void_p), ("scale_a", ctypes.c_void_p),
                ("codes_b", ctypes.c_void_p), ("scale_b", ctypes.c_void_p),
                ("acc", ctypes.c_void_p)]


class _Output(ctypes.Structure):
    _fields_ = [("accumulate", ctypes.c_int32), ("out_bf16", ctypes.c_int32), ("q", ctypes.POINTER(_QSpec)),
                ("step", ctypes.c_void_p), ("codes", ctypes.c_void_p), ("ld_codes", ctypes.c_int64),
                ("absmax", ctypes.c_void_p), ("raw_sums", ctypes.c_int32)]


@dataclass
class QSpec:
    """One quantization point (bits, scale mode, rounding mode, seed, tensor_id, index_offset, grid)."""
    bits: int = 8
    scale: int = PER_TENSOR
    round: int = SR
    seed: int = 0
    tensor_id: int = 0
    index_offset: int = 0
    format: int = GRID_INT
    absmax: Optional[torch.Tensor] = None      # device float tensor of one element: known max |x| (per tensor)

    def c(self) -> _QSpec:
        return _QSpec(self.bits, self.scale, self.round, self.format, self.seed, self.tensor_id,
                      self.index_offset, None if self.absmax is None else self.absmax.data_ptr())


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Loads libsrq.so (built in-tree by ``build.py``); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -m paper_2511_00874_b200.build` (there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
    qp = ctypes.POINTER(_QSpec)
    dp = ctypes.POINTER(_DebugOut)
    L.srq_quantize_workspace_bytes.argtypes = [i64, i64]
    L.srq_quantize_workspace_bytes.restype = sz
    L.srq_gemm_workspace_bytes.argtypes = [i64, i64]
    L.srq_gemm_workspace_bytes.restype = sz
    L.srq_workspace_bytes.argtypes = [i64, i64, i64]
    L.srq_workspace_bytes.restype = sz
    L.sr_quantize.argtypes = [vp, ctypes.c_int, i64, i64, i64, qp, vp, i64, vp, vp, i64, vp, vp, sz, vp]
    L.sr_quantize.restype = ctypes.c_int
    L.srq_absmax.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, vp]
    L.srq_absmax.restype = ctypes.c_int
    L.srq_absmax_cols.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, vp]
    L.srq_absmax_cols.restype = ctypes.c_int
    L.sr_quantize_static.argtypes = [vp, ctypes.c_int, i64, i64, i64, qp, vp, i64, vp, vp, i64, vp, vp, vp]
    L.sr_quantize_static.restype = ctypes.c_int
    L.srq_gemm_i8.argtypes = [vp, i64, vp, i64, i64, i64, i64, vp, i32, vp, i32, vp, i64, vp, vp, sz, vp]
    L.srq_gemm_i8.restype = ctypes.c_int
    L.srq_gemm_e4m3.argtypes = L.srq_gemm_i8.argtypes
    L.srq_gemm_e4m3.restype = ctypes.c_int
    for name in ("qlinear_fwd", "qlinear_bwd_input", "qlinear_bwd_weight"):
        f = getattr(L, name)
        f.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, qp, qp, vp, dp, vp, sz, vp]
        f.restype = ctypes.c_int
    L.qlinear_bwd.argtypes = [vp, vp, vp, ctypes.c_int, i64, i64, i64, qp, qp, qp, vp, vp, dp, dp, vp, sz, vp]
    L.qlinear_bwd.restype = ctypes.c_int
    op = ctypes.POINTER(_Output)
    L.srq_gemm_i8_ex.argtypes = [vp, i64, vp, i64, i64, i64, i64, vp, i32, vp, i32, vp, i64, vp, op, vp, sz, vp]
    L.srq_gemm_i8_ex.restype = ctypes.c_int
    L.qlinear_fwd_ex.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, qp, qp, vp, op, dp, vp, sz, vp]
    L.qlinear_fwd_ex.restype = ctypes.c_int
    L.qlinear_bwd_ex.argtypes = [vp, vp, vp, ctypes.c_int, i64, i64, i64, qp, qp, qp, vp, vp, op, op, dp, dp, vp, sz, vp]
    L.qlinear_bwd_ex.restype = ctypes.c_int
    L.srq_dequant_i32.argtypes = [vp, i64, i64, i64, vp, i32, vp, i32, vp, i64, i32, vp]
    L.srq_dequant_i32.restype = ctypes.c_int
    L.srq_selftest_bounded_wait.argtypes = [vp, sz, ctypes.c_uint32, vp]
    L.srq_selftest_bounded_wait.restype = ctypes.c_int
    L.srq_selftest_mma_rate.argtypes = [vp, sz, i32, ctypes.POINTER(i64), vp]
    L.srq_selftest_mma_rate.restype = ctypes.c_int
    L.srq_set_product_timer.argtypes = [vp, i64]
    L.srq_set_product_timer.restype = ctypes.c_int
    L.srq_plan_splits.argtypes = [i64, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.srq_plan_splits.restype = None
    L.srq_poll_status.argtypes = [vp, vp]
    L.srq_poll_status.restype = ctypes.c_int
    L.srq_status_string.argtypes = [ctypes.c_int]
    L.srq_status_string.restype = ctypes.c_char_p
    L.srq_launch_count.argtypes = []
    L.srq_launch_count.restype = ctypes.c_uint64
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().srq_status_string(int(status)).decode()


def launch_count() -> int:
    return int(lib().srq_launch_count())


def _check(status: int, where: str) -> None:
    if status != OK:
        raise SrqError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"inputs must be float32 or bfloat16, got {t.dtype}")


def _dev2d(t: torch.Tensor, name: str) -> None:
    if not t.is_cuda or t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{name} must be a 2-D CUDA tensor with unit inner stride")


def srq_quantize_workspace_bytes(rows: int, cols: int) -> int:
    return int(lib().srq_quantize_workspace_bytes(rows, cols))


def srq_gemm_workspace_bytes(M: int, N: int) -> int:
    return int(lib().srq_gemm_workspace_bytes(M, N))


def srq_workspace_bytes(T: int, N: int, K: int) -> int:
    return int(lib().srq_workspace_bytes(T, N, K))


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Device buffer for a workspace (torch's allocator returns 512-byte aligned blocks)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def sr_quantize(x: torch.Tensor, q: QSpec, codes_rm: Optional[torch.Tensor] = None,
                scale_rm: Optional[torch.Tensor] = None, codes_tr: Optional[torch.Tensor] = None,
                scale_tr: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None) -> None:
    """Def. 1-3 on x[rows, cols]; code tensors are int8 [rows, >=cols] / [cols, >=rows] views."""
    _dev2d(x, "x")
    rows, cols = x.shape
    if ws is None:
        ws = new_workspace(srq_quantize_workspace_bytes(rows, cols), x.device)
    cq = q.c()
    st = lib().sr_quantize(x.data_ptr(), _dtype_of(x), rows, cols, x.stride(0), ctypes.byref(cq),
                           _ptr(codes_rm), codes_rm.stride(0) if codes_rm is not None else 0,
                           _ptr(scale_rm),
                           _ptr(codes_tr), codes_tr.stride(0) if codes_tr is not None else 0,
                           _ptr(scale_tr), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "sr_quantize")


def srq_absmax(x: torch.Tensor, absmax: torch.Tensor) -> None:
    """max |x| into the one-element float32 CUDA tensor ``absmax``."""
    _dev2d(x, "x")
    st = lib().srq_absmax(x.data_ptr(), _dtype_of(x), x.shape[0], x.shape[1], x.stride(0), absmax.data_ptr(), _stream())
    _check(st, "srq_absmax")


def srq_absmax_cols(x: torch.Tensor, absmax_cols: torch.Tensor) -> None:
    """max |x[:, c]| of every column into the float32 CUDA tensor ``absmax_cols`` ([cols])."""
    _dev2d(x, "x")
    if absmax_cols.numel() < x.shape[1] or absmax_cols.dtype != torch.float32:
        raise ValueError("absmax_cols must hold cols float32 values")
    st = lib().srq_absmax_cols(x.data_ptr(), _dtype_of(x), x.shape[0], x.shape[1], x.stride(0), absmax_cols.data_ptr(), _stream())
    _check(st, "srq_absmax_cols")


def sr_quantize_static(x: torch.Tensor, q: QSpec, codes_rm: Optional[torch.Tensor] = None,
                       scale_rm: Optional[torch.Tensor] = None, codes_tr: Optional[torch.Tensor] = None,
                       scale_tr: Optional[torch.Tensor] = None,
                       device_status: Optional[torch.Tensor] = None) -> None:
    """sr_quantize without a workspace, for callers that must not allocate device memory: the
    scratch is the library's built-in 1 MiB array (shared by all calls on the device, so calls
    that may overlap must be ordered).  ``device_status`` is an optional int32 CUDA tensor of
    one element that receives the device-side status."""
    _dev2d(x, "x")
    rows, cols = x.shape
    cq = q.c()
    st = lib().sr_quantize_static(x.data_ptr(), _dtype_of(x), rows, cols, x.stride(0), ctypes.byref(cq),
                                  _ptr(codes_rm), codes_rm.stride(0) if codes_rm is not None else 0,
                                  _ptr(scale_rm),
                                  _ptr(codes_tr), codes_tr.stride(0) if codes_tr is not None else 0,
                                  _ptr(scale_tr), _ptr(device_status), _stream())
    _check(st, "sr_quantize_static")


def srq_gemm_i8(a: torch.Tensor, b: torch.Tensor, s_row: torch.Tensor, s_col: torch.Tensor,
                out: torch.Tensor, acc_out: Optional[torch.Tensor] = None,
                ws: Optional[torch.Tensor] = None) -> None:
    """out[M,N] = float(a[M,Kc] . b[N,Kc]^T) * (s_row x s_col); a, b int8 with pitch % 16 == 0."""
    _dev2d(a, "a")
    _dev2d(b, "b")
    M, Kc = a.shape
    N = b.shape[0]
    if ws is None:
        ws = new_workspace(srq_gemm_workspace_bytes(M, N), a.device)
    st = lib().srq_gemm_i8(a.data_ptr(), a.stride(0), b.data_ptr(), b.stride(0), M, N, Kc,
                           s_row.data_ptr(), int(s_row.numel() != 1), s_col.data_ptr(),
                           int(s_col.numel() != 1), out.data_ptr(), out.stride(0), _ptr(acc_out),
                           ws.data_ptr(), ws.numel(), _stream())
    _check(st, "srq_gemm_i8")


def srq_gemm_e4m3(a: torch.Tensor, b: torch.Tensor, s_row: torch.Tensor, s_col: torch.Tensor,
                  out: torch.Tensor, acc_out: Optional[torch.Tensor] = None,
                  ws: Optional[torch.Tensor] = None) -> None:
    """srq_gemm_i8 for E4M3 code bytes (uint8 tensors); acc_out, if given, is float32 [M, N]."""
    _dev2d(a, "a")
    _dev2d(b, "b")
    M, Kc = a.shape
    N = b.shape[0]
    if ws is None:
        ws = new_workspace(256, a.device)
    st = lib().srq_gemm_e4m3(a.data_ptr(), a.stride(0), b.data_ptr(), b.stride(0), M, N, Kc,
                             s_row.data_ptr(), int(s_row.numel() != 1), s_col.data_ptr(),
                             int(s_col.numel() != 1), out.data_ptr(), out.stride(0), _ptr(acc_out),
                             ws.data_ptr(), ws.numel(), _stream())
    _check(st, "srq_gemm_e4m3")


@dataclass
class DebugOut:
    """Optional device tensors that receive what a layer pass fed to its product."""
    codes_a: Optional[torch.Tensor] = None
    scale_a: Optional[torch.Tensor] = None
    codes_b: Optional[torch.Tensor] = None
    scale_b: Optional[torch.Tensor] = None
    acc: Optional[torch.Tensor] = None

    def c(self) -> _DebugOut:
        return _DebugOut(_ptr(self.codes_a), _ptr(self.scale_a), _ptr(self.codes_b),
                         _ptr(self.scale_b), _ptr(self.acc))


def _layer(fn_name: str, X0: torch.Tensor, X1: torch.Tensor, T: int, N: int, K: int, q0: QSpec,
           q1: QSpec, out: torch.Tensor, dbg: Optional[DebugOut], ws: Optional[torch.Tensor]) -> None:
    for t, n in ((X0, "first operand"), (X1, "second operand")):
        _dev2d(t, n)
        if not t.is_contiguous():
            raise ValueError(f"{n} must be contiguous")
    if _dtype_of(X0) != _dtype_of(X1):
        raise TypeError("both operands must have the same dtype")
    if out.dtype != torch.float32 or not out.is_contiguous():
        raise TypeError("output must be a contiguous float32 tensor")
    if ws is None:
        ws = new_workspace(srq_workspace_bytes(T, N, K), X0.device)
    c0, c1 = q0.c(), q1.c()
    cd = dbg.c() if dbg is not None else None
    st = getattr(lib(), fn_name)(X0.data_ptr(), X1.data_ptr(), _dtype_of(X0), T, N, K,
                                 ctypes.byref(c0), ctypes.byref(c1), out.data_ptr(),
                                 ctypes.byref(cd) if cd is not None else None,
                                 ws.data_ptr(), ws.numel(), _stream())
    _check(st, fn_name)


def qlinear_fwd(A: torch.Tensor, W: torch.Tensor, qA: QSpec, qW: QSpec, Y: torch.Tensor,
                dbg: Optional[DebugOut] = None, ws: Optional[torch.Tensor] = None) -> None:
    """Alg. 1: Y[T,N] = Q(A[T,K]) Q(W[N,K])^T."""
    T, K = A.shape
    N, K2 = W.shape
    if K != K2 or tuple(Y.shape) != (T, N):
        raise ValueError("qlinear_fwd: shapes must be A[T,K], W[N,K], Y[T,N]")
    _layer("qlinear_fwd", A, W, T, N, K, qA, qW, Y, dbg, ws)


def qlinear_bwd_input(dY: torch.Tensor, W: torch.Tensor, qdY: QSpec, qW: QSpec, dA: torch.Tensor,
                      dbg: Optional[DebugOut] = None, ws: Optional[torch.Tensor] = None) -> None:
    """Alg. 2: dA[T,K] = Q(dY[T,N]) Q(W[N,K])."""
    T, N = dY.shape
    N2, K = W.shape
    if N != N2 or tuple(dA.shape) != (T, K):
        raise ValueError("qlinear_bwd_input: shapes must be dY[T,N], W[N,K], dA[T,K]")
    _layer("qlinear_bwd_input", dY, W, T, N, K, qdY, qW, dA, dbg, ws)


def qlinear_bwd_weight(dY: torch.Tensor, A: torch.Tensor, qdY: QSpec, qA: QSpec, dW: torch.Tensor,
                       dbg: Optional[DebugOut] = None, ws: Optional[torch.Tensor] = None) -> None:
    """Alg. 2: dW[N,K] = Q(dY[T,N])^T Q(A[T,K])."""
    T, N = dY.shape
    T2, K = A.shape
    if T != T2 or tuple(dW.shape) != (N, K):
        raise ValueError("qlinear_bwd_weight: shapes must be dY[T,N], A[T,K], dW[N,K]")
    _layer("qlinear_bwd_weight", dY, A, T, N, K, qdY, qA, dW, dbg, ws)


def qlinear_bwd(dY: torch.Tensor, A: torch.Tensor, W: torch.Tensor, qdY: QSpec, qA: QSpec, qW: QSpec,
                dA: torch.Tensor, dW: torch.Tensor, dbg_input: Optional[DebugOut] = None,
                dbg_weight: Optional[DebugOut] = None, ws: Optional[torch.Tensor] = None) -> None:
    """Alg. 2 in one call: dA[T,K] = Q(dY) Q(W), dW[N,K] = Q(dY)^T Q(A); dY is read once."""
    T, N = dY.shape
    T2, K = A.shape
    N2, K2 = W.shape
    if T != T2 or N != N2 or K != K2 or tuple(dA.shape) != (T, K) or tuple(dW.shape) != (N, K):
        raise ValueError("qlinear_bwd: shapes must be dY[T,N], A[T,K], W[N,K], dA[T,K], dW[N,K]")
    for t, n in ((dY, "dY"), (A, "A"), (W, "W")):
        _dev2d(t, n)
        if not t.is_contiguous():
            raise ValueError(f"{n} must be contiguous")
    if not (_dtype_of(dY) == _dtype_of(A) == _dtype_of(W)):
        raise TypeError("all operands must have the same dtype")
    for t in (dA, dW):
        if t.dtype != torch.float32 or not t.is_contiguous():
            raise TypeError("outputs must be contiguous float32 tensors")
    if ws is None:
        ws = new_workspace(srq_workspace_bytes(T, N, K), dY.device)
    c0, c1, c2 = qdY.c(), qA.c(), qW.c()
    d0 = dbg_input.c() if dbg_input is not None else None
    d1 = dbg_weight.c() if dbg_weight is not None else None
    st = lib().qlinear_bwd(dY.data_ptr(), A.data_ptr(), W.data_ptr(), _dtype_of(dY), T, N, K,
                           ctypes.byref(c0), ctypes.byref(c1), ctypes.byref(c2), dA.data_ptr(), dW.data_ptr(),
                           ctypes.byref(d0) if d0 is not None else None,
                           ctypes.byref(d1) if d1 is not None else None,
                           ws.data_ptr(), ws.numel(), _stream())
    _check(st, "qlinear_bwd")


@dataclass
class Output:
    """Output options of a product (srq_output_t): accumulate into out, codes of Q(result) with a
    caller-supplied step (q, step, codes), absmax of the result.  A bfloat16 output tensor passed
    to one of the *_ex calls sets the struct's out_bf16 member."""
    accumulate: int = 0        # 1 (or True): out += result in binary32; 2: running int32 sums in acc_out
    q: Optional[QSpec] = None
    step: Optional[torch.Tensor] = None
    codes: Optional[torch.Tensor] = None
    absmax: Optional[torch.Tensor] = None

    def c(self, out_bf16: bool = False, raw_sums: bool = False):
        cq = self.q.c() if self.q is not None else None
        o = _Output(int(self.accumulate), int(out_bf16), ctypes.pointer(cq) if cq is not None else None, _ptr(self.step),
                    _ptr(self.codes), self.codes.stride(0) if self.codes is not None else 0, _ptr(self.absmax),
                    int(raw_sums))
        o._keep = cq                      # the struct points into cq
        return o


def _opt(o: Optional[Output], out: Optional[torch.Tensor] = None):
    """The C struct of the options; a bfloat16 output tensor selects out_bf16 by itself, an int32
    output tensor raw_sums (the exact sums, unscaled)."""
    bf16 = out is not None and out.dtype == torch.bfloat16
    raw = out is not None and out.dtype == torch.int32
    if out is not None and not bf16 and not raw and out.dtype != torch.float32:
        raise TypeError("the output of a product is float32, bfloat16 or (raw sums) int32")
    if o is None:
        return Output().c(bf16, raw) if (bf16 or raw) else None
    return o.c(bf16, raw)


def srq_gemm_i8_ex(a: torch.Tensor, b: torch.Tensor, s_row: torch.Tensor, s_col: torch.Tensor,
                   out: Optional[torch.Tensor], output: Optional[Output] = None,
                   acc_out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None) -> None:
    """srq_gemm_i8 with output options; out may be None when codes are requested."""
    _dev2d(a, "a")
    _dev2d(b, "b")
    M, Kc = a.shape
    N = b.shape[0]
    if ws is None:
        ws = new_workspace(srq_gemm_workspace_bytes(M, N), a.device)
    co = _opt(output, out)
    st = lib().srq_gemm_i8_ex(a.data_ptr(), a.stride(0), b.data_ptr(), b.stride(0), M, N, Kc,
                              s_row.data_ptr(), int(s_row.numel() != 1), s_col.data_ptr(), int(s_col.numel() != 1),
                              _ptr(out), out.stride(0) if out is not None else 0, _ptr(acc_out),
                              ctypes.byref(co) if co is not None else None, ws.data_ptr(), ws.numel(), _stream())
    _check(st, "srq_gemm_i8_ex")


def qlinear_fwd_ex(A: torch.Tensor, W: torch.Tensor, qA: QSpec, qW: QSpec, Y: Optional[torch.Tensor],
                   output: Optional[Output] = None, dbg: Optional[DebugOut] = None,
                   ws: Optional[torch.Tensor] = None) -> None:
    """qlinear_fwd with output options; Y may be None when codes are requested."""
    T, K = A.shape
    N = W.shape[0]
    if ws is None:
        ws = new_workspace(srq_workspace_bytes(T, N, K), A.device)
    c0, c1 = qA.c(), qW.c()
    cd = dbg.c() if dbg is not None else None
    co = _opt(output, Y)
    st = lib().qlinear_fwd_ex(A.data_ptr(), W.data_ptr(), _dtype_of(A), T, N, K, ctypes.byref(c0), ctypes.byref(c1),
                              _ptr(Y), ctypes.byref(co) if co is not None else None,
                              ctypes.byref(cd) if cd is not None else None, ws.data_ptr(), ws.numel(), _stream())
    _check(st, "qlinear_fwd_ex")


def qlinear_bwd_ex(dY: torch.Tensor, A: torch.Tensor, W: torch.Tensor, qdY: QSpec, qA: QSpec, qW: QSpec,
                   dA: Optional[torch.Tensor], dW: Optional[torch.Tensor], output_dA: Optional[Output] = None,
                   output_dW: Optional[Output] = None, ws: Optional[torch.Tensor] = None,
                   dbg_input: Optional[DebugOut] = None, dbg_weight: Optional[DebugOut] = None) -> None:
    """qlinear_bwd with output options for dA and dW (dbg_weight.acc holds the running int32 sums of
    dW when output_dW.accumulate is 2)."""
    T, N = dY.shape
    K = A.shape[1]
    if ws is None:
        ws = new_workspace(srq_workspace_bytes(T, N, K), dY.device)
    c0, c1, c2 = qdY.c(), qA.c(), qW.c()
    o0, o1 = _opt(output_dA, dA), _opt(output_dW, dW)
    d0 = dbg_input.c() if dbg_input is not None else None
    d1 = dbg_weight.c() if dbg_weight is not None else None
    st = lib().qlinear_bwd_ex(dY.data_ptr(), A.data_ptr(), W.data_ptr(), _dtype_of(dY), T, N, K,
                              ctypes.byref(c0), ctypes.byref(c1), ctypes.byref(c2), _ptr(dA), _ptr(dW),
                              ctypes.byref(o0) if o0 is not None else None,
                              ctypes.byref(o1) if o1 is not None else None,
                              ctypes.byref(d0) if d0 is not None else None,
                              ctypes.byref(d1) if d1 is not None else None,
                              ws.data_ptr(), ws.numel(), _stream())
    _check(st, "qlinear_bwd_ex")


def srq_dequant_i32(acc: torch.Tensor, s_row: torch.Tensor, s_col: torch.Tensor, out: torch.Tensor) -> None:
    """out[M,N] = float(acc[M,N]) * (s_row x s_col): the finishing step over int32 sums (e.g. the
    all-reduced raw sums of token shards).  out is float32 or bfloat16."""
    _dev2d(acc, "acc")
    _dev2d(out, "out")
    if acc.dtype != torch.int32 or out.dtype not in (torch.float32, torch.bfloat16) or acc.shape != out.shape:
        raise TypeError("acc must be int32 [M, N], out float32 or bfloat16 [M, N]")
    M, N = acc.shape
    st = lib().srq_dequant_i32(acc.data_ptr(), acc.stride(0), M, N, s_row.data_ptr(), int(s_row.numel() != 1),
                               s_col.data_ptr(), int(s_col.numel() != 1), out.data_ptr(), out.stride(0),
                               int(out.dtype == torch.bfloat16), _stream())
    _check(st, "srq_dequant_i32")


def srq_plan_splits(tiles: int, k_blocks: int, groups: int):
    """(full_tiles, splits) the product kernel would use (host-side rule, no device needed)."""
    f, s = ctypes.c_int32(), ctypes.c_int32()
    lib().srq_plan_splits(tiles, k_blocks, groups, ctypes.byref(f), ctypes.byref(s))
    return f.value, s.value


def srq_selftest_bounded_wait(ws: torch.Tensor, limit_us: int = 1000) -> None:
    """Enqueues the bounded-wait self-test; srq_poll_status(ws) then returns ERR_TIMEOUT."""
    _check(lib().srq_selftest_bounded_wait(ws.data_ptr(), ws.numel(), int(limit_us), _stream()), "srq_selftest_bounded_wait")


def srq_selftest_mma_rate(ws: torch.Tensor, k_blocks: int) -> int:
    """Enqueues the tensor-pipe issue-rate microbenchmark (operands resident in shared memory, no
    global traffic); returns the integer operations of the launch.  Time it with CUDA events."""
    ops = ctypes.c_int64(0)
    _check(lib().srq_selftest_mma_rate(ws.data_ptr(), ws.numel(), int(k_blocks), ctypes.byref(ops), _stream()),
           "srq_selftest_mma_rate")
    return int(ops.value)


def srq_set_product_timer(slots: Optional[torch.Tensor]) -> None:
    """Device-side start / end times (ns) of the next product launches into ``slots``, an int64 CUDA
    tensor of shape [n, 2] initialised with ``new_product_timer``; None switches the timing off."""
    if slots is None:
        _check(lib().srq_set_product_timer(None, 0), "srq_set_product_timer")
        return
    if slots.dtype != torch.int64 or slots.dim() != 2 or slots.shape[1] != 2 or not slots.is_contiguous():
        raise TypeError("slots must be a contiguous int64 CUDA tensor of shape [n, 2]")
    _check(lib().srq_set_product_timer(slots.data_ptr(), slots.shape[0]), "srq_set_product_timer")


def new_product_timer(n: int, device="cuda") -> torch.Tensor:
    """[n, 2] slots holding (all ones, zero): what srq_set_product_timer expects."""
    t = torch.zeros((n, 2), dtype=torch.int64, device=device)
    t[:, 0] = -1
    return t


def srq_poll_status(ws: torch.Tensor) -> int:
    """Synchronises the current stream and returns the device status word of ``ws``."""
    return int(lib().srq_poll_status(ws.data_ptr(), _stream()))
