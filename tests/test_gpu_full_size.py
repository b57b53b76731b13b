"""Parity at the full size and launch configuration of the benchmark and of every layer shape of the
GPT-2-small and Llama-style workload families.

Linear layer 4096 -> 4096 with 65536 tokens, fp32 inputs, 8-bit per-tensor SR: the workload
`bench.py` times, called the way it calls it (no debug copies, so the products run as CTA pairs
and store their results as whole blocks); and the largest layer of the per-row configuration
(2048 -> 5632, 65536 tokens, bf16 inputs, 8-bit forward, 4-bit backward).  The oracle cannot form 3 x 1.1e12 products in a test,
so the comparison is:
  - every int8 code and step size of all operands against the oracle's quantizer (bit for bit);
  - sampled rows of Y, dA and dW against oracle products of the oracle's codes (bit for bit);
  - the whole of every output against a second GPU path (the product on the same codes with raw
    sums requested, which stores element-wise) and that path's int32 sums against exact
    Freivalds products  acc r == qa (qb^T r)  evaluated in binary64, where they are exact.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import synth

pytestmark = pytest.mark.gpu


def _oq(q):
    return oracle.QSpec(q.bits, q.scale, q.round, q.seed, q.tensor_id, q.index_offset)


def _codes(x, q, rm, tr):
    rows, cols = x.shape
    per_row = q.scale == srq.PER_ROW
    crm = torch.empty((rows, cols), dtype=torch.int8, device="cuda") if rm else None
    ctr = torch.empty((cols, rows), dtype=torch.int8, device="cuda") if tr else None
    s1 = torch.empty(rows if per_row else 1, device="cuda")
    s2 = torch.empty(cols if per_row else 1, device="cuda")
    srq.sr_quantize(x, q, crm, s1 if rm else None, ctr, s2 if tr else None)
    return crm, ctr, s1 if rm else None, s2 if tr else None


def _freivalds(acc, qa, qb, rng):
    """acc[M,N] == qa[M,Kc] qb[N,Kc]^T checked with random small-integer vectors, exactly."""
    accd = acc.double()
    for _ in range(2):
        r = torch.from_numpy(rng.integers(-3, 4, (qb.shape[0], 1)).astype(np.float64)).cuda()
        # chunked so that the binary64 copies of the code matrices stay small
        right = torch.zeros((qb.shape[1], 1), dtype=torch.float64, device="cuda")
        for j in range(0, qb.shape[0], 4096):
            right += qb[j:j + 4096].double().t() @ r[j:j + 4096]
        lhs = accd @ r
        for i in range(0, qa.shape[0], 8192):
            assert torch.equal(lhs[i:i + 8192], qa[i:i + 8192].double() @ right)


CASES = {
    # the benchmark workload: linear 4096 -> 4096, fp32, 8-bit per-tensor SR
    "bench": (65536, 4096, 4096, torch.float32, srq.PER_TENSOR, 8, 8),
    # the largest Llama-style layer of the per-row configuration: bf16, 8-bit forward, 4-bit backward
    "gate_up": (65536, 5632, 2048, torch.bfloat16, srq.PER_ROW, 8, 4),
    # every other layer shape the workload families name, at its largest token count: other tile
    # counts, split plans and tails (2304 = 9 x 256 columns, a 5632-long contraction, 768-wide outputs
    # whose weight gradient splits the contraction over all CTA pairs)
    "gpt2_qkv": (65536, 2304, 768, torch.float32, srq.PER_TENSOR, 8, 8),
    "gpt2_proj": (65536, 768, 768, torch.float32, srq.PER_TENSOR, 8, 8),
    "gpt2_fc1": (65536, 3072, 768, torch.float32, srq.PER_TENSOR, 8, 8),
    "gpt2_fc2": (65536, 768, 3072, torch.float32, srq.PER_TENSOR, 8, 8),
    "llama_qkv": (65536, 2560, 2048, torch.bfloat16, srq.PER_ROW, 8, 4),
    "llama_o": (65536, 2048, 2048, torch.bfloat16, srq.PER_ROW, 8, 4),
    "llama_down": (65536, 2048, 5632, torch.bfloat16, srq.PER_ROW, 8, 4),
}


@pytest.mark.parametrize("case", list(CASES))
def test_layer_at_full_size(case):
    T, N, K, dtype, scale, bits_f, bits_b = CASES[case]
    A = synth.normal((T, K), 1.0, 1000, dtype, "cuda")
    dY = synth.normal((T, N), 1e-3, 1001, dtype, "cuda")
    W = synth.normal((N, K), 0.02, 7, dtype, "cuda")
    bits = {"a_f": bits_f, "w_f": bits_f, "a_b": bits_b, "w_b": bits_b, "dy": bits_b}
    q = {k: srq.QSpec(bits[k], scale, srq.SR, 3, i) for i, k in enumerate(["a_f", "w_f", "a_b", "w_b", "dy"])}
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    Y = torch.empty((T, N), device="cuda")
    dA = torch.empty((T, K), device="cuda")
    dW = torch.empty((N, K), device="cuda")
    srq.qlinear_fwd(A, W, q["a_f"], q["w_f"], Y, None, ws)
    srq.qlinear_bwd(dY, A, W, q["dy"], q["a_b"], q["w_b"], dA, dW, None, None, ws)
    assert srq.srq_poll_status(ws) == 0

    # ---- codes and step sizes of every operand, whole tensors, against the oracle
    hA, hW, hdY = A.float().cpu().numpy(), W.float().cpu().numpy(), dY.float().cpu().numpy()
    o_af = oracle.sr_quantize(hA, _oq(q["a_f"]), True, False)
    o_wf = oracle.sr_quantize(hW, _oq(q["w_f"]), True, False)
    o_dy = oracle.sr_quantize(hdY, _oq(q["dy"]), True, True)
    o_wb = oracle.sr_quantize(hW, _oq(q["w_b"]), False, True)
    o_ab = oracle.sr_quantize(hA, _oq(q["a_b"]), False, True)
    g_af, _, s_af, _ = _codes(A, q["a_f"], True, False)
    g_wf, _, s_wf, _ = _codes(W, q["w_f"], True, False)
    g_dy, g_dyt, s_dy, s_dyt = _codes(dY, q["dy"], True, True)
    _, g_wbt, _, s_wb = _codes(W, q["w_b"], False, True)
    _, g_abt, _, s_ab = _codes(A, q["a_b"], False, True)
    for name, g, o in (("A fwd", g_af, o_af[0]), ("W fwd", g_wf, o_wf[0]), ("dY", g_dy, o_dy[0]),
                       ("dY^T", g_dyt, o_dy[2]), ("W^T bwd", g_wbt, o_wb[2]), ("A^T bwd", g_abt, o_ab[2])):
        assert np.array_equal(g.cpu().numpy(), o), name + ": codes"
    for name, g, o in (("A fwd", s_af, o_af[1]), ("W fwd", s_wf, o_wf[1]), ("dY", s_dy, o_dy[1]), ("dY^T", s_dyt, o_dy[3]),
                       ("W bwd", s_wb, o_wb[3]), ("A bwd", s_ab, o_ab[3])):
        assert np.array_equal(g.cpu().numpy(), o), name + ": step size"

    # ---- sampled rows of the three outputs against oracle products of the oracle's codes
    rng = np.random.default_rng(0)
    rows_t = np.sort(rng.choice(T, 48, replace=False))
    rows_n = np.sort(rng.choice(N, 12, replace=False))
    pick = lambda sc, rows: sc if sc.size == 1 else sc[rows]
    ref = oracle.dequant(oracle.gemm_i8_nt(o_af[0][rows_t], o_wf[0]), pick(o_af[1], rows_t), o_wf[1])
    assert np.array_equal(Y[torch.from_numpy(rows_t).cuda()].cpu().numpy(), ref), "Y rows"
    ref = oracle.dequant(oracle.gemm_i8_nt(o_dy[0][rows_t], o_wb[2]), pick(o_dy[1], rows_t), o_wb[3])
    assert np.array_equal(dA[torch.from_numpy(rows_t).cuda()].cpu().numpy(), ref), "dA rows"
    ref = oracle.dequant(oracle.gemm_i8_nt(o_dy[2][rows_n], o_ab[2]), pick(o_dy[3], rows_n), o_ab[3])
    assert np.array_equal(dW[torch.from_numpy(rows_n).cuda()].cpu().numpy(), ref), "dW rows"
    del hA, hW, hdY, o_af, o_wf, o_dy, o_wb, o_ab

    # ---- whole outputs: the element-wise path on the same codes gives the same values, and its
    # int32 sums pass exact Freivalds checks
    gws = srq.new_workspace(srq.srq_gemm_workspace_bytes(max(T, N), max(N, K)))
    for name, qa, qb, sa, sb, out in (("Y", g_af, g_wf, s_af, s_wf, Y), ("dA", g_dy, g_wbt, s_dy, s_wb, dA),
                                      ("dW", g_dyt, g_abt, s_dyt, s_ab, dW)):
        acc = torch.empty(out.shape, dtype=torch.int32, device="cuda")
        out2 = torch.empty_like(out)
        srq.srq_gemm_i8(qa, qb, sa, sb, out2, acc, gws)
        assert srq.srq_poll_status(gws) == 0
        assert torch.equal(out2, out), name + ": block-store path differs from the element-wise path"
        _freivalds(acc, qa, qb, rng)
        del acc, out2


@pytest.mark.parametrize("scale,dtype", [(srq.PER_TENSOR, torch.float32), (srq.PER_ROW, torch.bfloat16)])
def test_layer_on_the_floating_point_grid_over_many_tiles(scale, dtype):
    """The E4M3 grid at a size that runs many rounds of CTA-pair tiles (16384 tokens, 4096 -> 4096):
    every code and step size of all five quantization points against the oracle (bit for bit), and
    sampled rows of Y, dA and dW against the oracle's exact binary64 products of those codes within
    1e-5 * |row| * |col| (the summation order of the binary32 accumulators is the hardware's)."""
    T, N, K = 16384, 4096, 4096
    A = synth.normal((T, K), 1.0, 2000, dtype, "cuda")
    dY = synth.normal((T, N), 1e-3, 2001, dtype, "cuda")
    W = synth.normal((N, K), 0.02, 2002, dtype, "cuda")
    q = {k: srq.QSpec(8, scale, srq.SR, 4, i, 0, srq.GRID_E4M3) for i, k in enumerate(["a_f", "w_f", "a_b", "w_b", "dy"])}
    oq = lambda s: oracle.QSpec(s.bits, s.scale, s.round, s.seed, s.tensor_id, s.index_offset)
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    Y, dA, dW = torch.empty((T, N), device="cuda"), torch.empty((T, K), device="cuda"), torch.empty((N, K), device="cuda")
    srq.qlinear_fwd(A, W, q["a_f"], q["w_f"], Y, None, ws)
    srq.qlinear_bwd(dY, A, W, q["dy"], q["a_b"], q["w_b"], dA, dW, None, None, ws)
    assert srq.srq_poll_status(ws) == 0
    hA, hW, hdY = A.float().cpu().numpy(), W.float().cpu().numpy(), dY.float().cpu().numpy()
    o_af = oracle.sr_quantize_e4m3(hA, oq(q["a_f"]), True, False)
    o_wf = oracle.sr_quantize_e4m3(hW, oq(q["w_f"]), True, False)
    o_dy = oracle.sr_quantize_e4m3(hdY, oq(q["dy"]), True, True)
    o_wb = oracle.sr_quantize_e4m3(hW, oq(q["w_b"]), False, True)
    o_ab = oracle.sr_quantize_e4m3(hA, oq(q["a_b"]), False, True)
    g_af = _codes(A, q["a_f"], True, False)
    g_wf = _codes(W, q["w_f"], True, False)
    g_dy = _codes(dY, q["dy"], True, True)
    g_wb = _codes(W, q["w_b"], False, True)
    g_ab = _codes(A, q["a_b"], False, True)
    u8 = lambda t: t.view(torch.uint8).cpu().numpy()
    for name, g, o in (("A fwd", g_af[0], o_af[0]), ("W fwd", g_wf[0], o_wf[0]), ("dY", g_dy[0], o_dy[0]), ("dY^T", g_dy[1], o_dy[2]),
                       ("W^T bwd", g_wb[1], o_wb[2]), ("A^T bwd", g_ab[1], o_ab[2])):
        assert np.array_equal(u8(g), o), name + ": codes"
    for name, g, o in (("A fwd", g_af[2], o_af[1]), ("W fwd", g_wf[2], o_wf[1]), ("dY", g_dy[2], o_dy[1]), ("dY^T", g_dy[3], o_dy[3]),
                       ("W bwd", g_wb[3], o_wb[3]), ("A bwd", g_ab[3], o_ab[3])):
        assert np.array_equal(g.cpu().numpy(), o), name + ": step size"
    rng = np.random.default_rng(1)
    rows_t = np.sort(rng.choice(T, 24, replace=False))
    rows_n = np.sort(rng.choice(N, 8, replace=False))
    pick = lambda sc, rows: sc if sc.size == 1 else sc[rows]

    def check(name, out, rows, ca, sa, cb, sb):
        _, ref = oracle.gemm_e4m3_nt(ca[rows], cb, pick(sa, rows), sb)
        na = np.linalg.norm(oracle.e4m3_decode(ca[rows]), axis=1)
        nb = np.linalg.norm(oracle.e4m3_decode(cb), axis=1)
        sc = np.broadcast_to(pick(sa, rows), (len(rows),))[:, None].astype(np.float64) * np.broadcast_to(sb, (cb.shape[0],))[None, :]
        bound = 1e-5 * na[:, None] * nb[None, :] * sc + 1e-30
        got = out[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= bound * 1.001 + np.abs(ref) * 2e-7), name

    check("Y rows", Y, rows_t, o_af[0], o_af[1], o_wf[0], o_wf[1])
    check("dA rows", dA, rows_t, o_dy[0], o_dy[1], o_wb[2], o_wb[3])
    check("dW rows", dW, rows_n, o_dy[2], o_dy[3], o_ab[2], o_ab[3])
