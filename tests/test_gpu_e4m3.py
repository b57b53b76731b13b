"""GPU parity of the E4M3 path: code bytes and step sizes bit for bit against the oracle; products
within 1e-5 * |row| * |col| of the oracle's exact sums (binary32 accumulation on the tensor cores
has an order of its own, so the sums cannot be compared bit for bit)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _q(scale, rnd, seed=0, tid=0, off=0, bits=8):
    return srq.QSpec(bits, scale, rnd, seed, tid, off, srq.GRID_E4M3)


def _oq(q):
    return oracle.QSpec(q.bits, q.scale, q.round, q.seed, q.tensor_id, q.index_offset)


def _quantize_gpu(x, q, want_rm=True, want_tr=True):
    rows, cols = x.shape
    per_row = q.scale == srq.PER_ROW
    crm = torch.full((rows, cols), 99, dtype=torch.int8, device="cuda") if want_rm else None
    ctr = torch.full((cols, rows), 99, dtype=torch.int8, device="cuda") if want_tr else None
    srm = torch.empty(rows if per_row else 1, device="cuda") if want_rm else None
    stt = torch.empty(cols if per_row else 1, device="cuda") if want_tr else None
    ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(rows, cols))
    srq.sr_quantize(x, q, crm, srm, ctr, stt, ws)
    assert srq.srq_poll_status(ws) == 0
    f = lambda t: None if t is None else t.cpu().numpy()
    u = lambda t: None if t is None else t.view(torch.uint8).cpu().numpy()
    return u(crm), f(srm), u(ctr), f(stt)


def _check_quantizer(x, q):
    got = _quantize_gpu(x, q)
    ref = oracle.sr_quantize_e4m3(x.float().cpu().numpy(), _oq(q), True, True)
    for name, g, r in zip(("codes_rm", "scale_rm", "codes_tr", "scale_tr"), got, ref):
        bad = np.argwhere(g != r)
        assert bad.size == 0, f"{name}: {len(bad)} mismatches, first at {bad[0]}: gpu {g[tuple(bad[0])]} oracle {r[tuple(bad[0])]}"


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
@pytest.mark.parametrize("rnd", [srq.SR, srq.RTN])
def test_codes_match_the_oracle_on_tiles_with_a_ragged_tail(dtype, scale, rnd):
    x = synth.with_outliers((300, 388), seed=3, dtype=dtype, device="cuda")
    _check_quantizer(x, _q(scale, rnd, seed=5, tid=9))


@pytest.mark.parametrize("shape,off", [((131, 259), 0), ((17, 5), 3), ((1, 1), 0), ((129, 130), 2 ** 33 + 2)])
def test_codes_match_on_unaligned_extents_and_offsets(shape, off):
    x = synth.normal(shape, 1.0, seed=shape[0], device="cuda")
    for scale in (srq.PER_TENSOR, srq.PER_ROW):
        _check_quantizer(x, _q(scale, srq.SR, seed=2 ** 40 + 3, tid=2 ** 35 + 1, off=off))
        _check_quantizer(x, _q(scale, srq.RTN))


def test_wide_dynamic_range_zero_groups_and_grid_values():
    # values across all binades and the subnormal range of the grid, a zero row and a zero column
    g = torch.Generator().manual_seed(1)
    x = (torch.randn(140, 132, generator=g) * torch.exp2(torch.randint(-14, 9, (140, 132), generator=g).float())).cuda()
    x[5] = 0
    x[:, 9] = 0
    x[0, 0] = 448.0
    for scale in (srq.PER_TENSOR, srq.PER_ROW):
        _check_quantizer(x, _q(scale, srq.SR, seed=1))
        _check_quantizer(x, _q(scale, srq.RTN))
    # every finite grid value, scaled by a power of two, is reproduced exactly
    codes = torch.tensor([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=torch.uint8)
    vals = (codes.view(torch.float8_e4m3fn).float() * 0.25).reshape(1, -1).cuda()
    got = _quantize_gpu(vals.contiguous(), _q(srq.PER_TENSOR, srq.SR, seed=4), True, False)
    back = torch.from_numpy(got[0]).view(torch.float8_e4m3fn).float() * float(got[1][0])
    assert torch.equal(back, vals.cpu())


def _finite_codes(rows, kc, seed):
    g = torch.Generator().manual_seed(seed)
    c = torch.randint(0, 256, (rows, (kc + 15) // 16 * 16), generator=g, dtype=torch.int32).to(torch.uint8)
    c[(c & 0x7F) == 0x7F] = 0x38          # no NaN codes
    return c.cuda()[:, :kc]


def _bound(a, b, s_row, s_col):
    """1e-5 * |row_i| * |col_j| (norms of the decoded code values), and the same times the scales."""
    na = np.linalg.norm(oracle.e4m3_decode(a), axis=1)
    nb = np.linalg.norm(oracle.e4m3_decode(b), axis=1)
    acc_b = TOL * na[:, None] * nb[None, :]
    sc = (np.broadcast_to(s_row, (a.shape[0],))[:, None] * np.broadcast_to(s_col, (b.shape[0],))[None, :]).astype(np.float64)
    return acc_b, acc_b * sc + 1e-30


@pytest.mark.parametrize("M,N,Kc", [(64, 256, 256), (1, 1, 1), (129, 257, 130), (300, 520, 1000), (384, 768, 4096)])
@pytest.mark.parametrize("per_row", [False, True])
def test_product_within_the_accumulation_bound(M, N, Kc, per_row):
    a, b = _finite_codes(M, Kc, 1), _finite_codes(N, Kc, 2)
    s_row = (torch.rand(M if per_row else 1) * 0.1 + 1e-3).cuda()
    s_col = (torch.rand(N if per_row else 1) * 0.1 + 1e-3).cuda()
    ha, hb = a.cpu().numpy(), b.cpu().numpy()
    ref_acc, ref_out = oracle.gemm_e4m3_nt(ha, hb, s_row.cpu().numpy(), s_col.cpu().numpy())
    acc_b, out_b = _bound(ha, hb, s_row.cpu().numpy(), s_col.cpu().numpy())
    for want_acc in (True, False):          # element-wise epilogue, then block stores
        out = torch.full((M, N), float("nan"), device="cuda")
        acc = torch.full((M, N), float("nan"), device="cuda") if want_acc else None
        ws = srq.new_workspace(256)
        srq.srq_gemm_e4m3(a, b, s_row, s_col, out, acc, ws)
        assert srq.srq_poll_status(ws) == 0
        if want_acc:
            assert np.all(np.abs(acc.cpu().numpy().astype(np.float64) - ref_acc) <= acc_b)
        assert np.all(np.abs(out.cpu().numpy().astype(np.float64) - ref_out) <= out_b * 1.001 + np.abs(ref_out) * 2e-7)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
def test_layer_passes_on_the_e4m3_grid(dtype, scale):
    T, N, K = 264, 392, 328
    A, W, dY = synth.layer_inputs(T, N, K, seed=1, dtype=dtype, device="cuda", std_dy=1e-3)
    q = {k: _q(scale, srq.SR, seed=3, tid=i) for i, k in enumerate(["a_f", "w_f", "a_b", "w_b", "dy"])}
    f = lambda t: t.float().cpu().numpy()
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    cases = [("fwd", srq.qlinear_fwd, oracle.qlinear_fwd_e4m3, A, W, q["a_f"], q["w_f"], (T, K), (N, K), (T, N)),
             ("bwd_input", srq.qlinear_bwd_input, oracle.qlinear_bwd_input_e4m3, dY, W, q["dy"], q["w_b"], (T, N), (K, N), (T, K)),
             ("bwd_weight", srq.qlinear_bwd_weight, oracle.qlinear_bwd_weight_e4m3, dY, A, q["dy"], q["a_b"], (N, T), (K, T), (N, K))]
    outs = {}
    for name, fn, ofn, X0, X1, q0, q1, sa, sb, so in cases:
        per_row = scale == srq.PER_ROW
        out = torch.full(so, float("nan"), device="cuda")
        dbg = srq.DebugOut(torch.empty(sa, dtype=torch.int8, device="cuda"), torch.empty(sa[0] if per_row else 1, device="cuda"),
                           torch.empty(sb, dtype=torch.int8, device="cuda"), torch.empty(sb[0] if per_row else 1, device="cuda"), None)
        fn(X0, X1, q0, q1, out, dbg, ws)
        assert srq.srq_poll_status(ws) == 0
        ref = ofn(f(X0), f(X1), _oq(q0), _oq(q1))
        assert np.array_equal(dbg.codes_a.view(torch.uint8).cpu().numpy(), ref.codes_a), name + ": codes of first operand"
        assert np.array_equal(dbg.codes_b.view(torch.uint8).cpu().numpy(), ref.codes_b), name + ": codes of second operand"
        assert np.array_equal(dbg.scale_a.cpu().numpy(), ref.scale_a) and np.array_equal(dbg.scale_b.cpu().numpy(), ref.scale_b)
        _, out_b = _bound(ref.codes_a, ref.codes_b, ref.scale_a, ref.scale_b)
        assert np.all(np.abs(out.cpu().numpy().astype(np.float64) - ref.out) <= out_b * 1.001 + np.abs(ref.out) * 2e-7), name
        outs[name] = out
    # Alg. 2 in one call gives the same outputs as the two separate calls (same kernels, same order)
    dA, dW = torch.empty((T, K), device="cuda"), torch.empty((N, K), device="cuda")
    srq.qlinear_bwd(dY, A, W, q["dy"], q["a_b"], q["w_b"], dA, dW, None, None, ws)
    assert srq.srq_poll_status(ws) == 0
    assert torch.equal(dA, outs["bwd_input"]) and torch.equal(dW, outs["bwd_weight"])


def test_operands_of_one_product_must_share_the_grid():
    A, W, _ = synth.layer_inputs(64, 64, 64, seed=2, device="cuda")
    Y = torch.empty((64, 64), device="cuda")
    with pytest.raises(srq.SrqError) as e:
        srq.qlinear_fwd(A, W, _q(srq.PER_TENSOR, srq.SR), srq.QSpec(8), Y)
    assert e.value.status == 1


@pytest.mark.parametrize("bits", [7, 6, 5])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_narrow_formats_e4m2_e4m1_e4m0(bits, dtype):
    """The E4M3 values with 2, 1, 0 mantissa bits: codes and step sizes bit for bit, both layouts,
    fast and general quantizer paths, the one-pass per-row kernel; every code has its low mantissa
    bits clear; the layer passes run on the same product as E4M3."""
    low = (1 << (8 - bits)) - 1
    for shape, off in (((300, 388), 0), ((131, 259), 3), ((40, 1024), 4)):
        x = synth.with_outliers(shape, seed=bits, dtype=dtype, device="cuda")
        x[1] = 0
        for scale in (srq.PER_TENSOR, srq.PER_ROW):
            for rnd in (srq.SR, srq.RTN):
                q = _q(scale, rnd, seed=6, tid=2 ** 33 + 1, off=off, bits=bits)
                _check_quantizer(x, q)
                crm = _quantize_gpu(x, q, True, False)[0]          # rows of 1024: one-pass per-row kernel
                assert not (crm & low).any()
                ref = oracle.sr_quantize_e4m3(x.float().cpu().numpy(), _oq(q), True, False)
                assert np.array_equal(crm, ref[0])
    T, N, K = 136, 264, 200
    A, W, dY = synth.layer_inputs(T, N, K, seed=2, dtype=dtype, device="cuda", std_dy=1e-3)
    qa, qw, qdy = (_q(srq.PER_ROW, srq.SR, seed=1, tid=i, bits=bits) for i in range(3))
    f = lambda t: t.float().cpu().numpy()
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    Y = torch.empty((T, N), device="cuda")
    dbg = srq.DebugOut(torch.empty((T, K), dtype=torch.int8, device="cuda"), torch.empty(T, device="cuda"),
                       torch.empty((N, K), dtype=torch.int8, device="cuda"), torch.empty(N, device="cuda"), None)
    srq.qlinear_fwd(A, W, qa, qw, Y, dbg, ws)
    assert srq.srq_poll_status(ws) == 0
    ref = oracle.qlinear_fwd_e4m3(f(A), f(W), _oq(qa), _oq(qw))
    assert np.array_equal(dbg.codes_a.view(torch.uint8).cpu().numpy(), ref.codes_a)
    assert np.array_equal(dbg.codes_b.view(torch.uint8).cpu().numpy(), ref.codes_b)
    _, out_b = _bound(ref.codes_a, ref.codes_b, ref.scale_a, ref.scale_b)
    assert np.all(np.abs(Y.cpu().numpy().astype(np.float64) - ref.out) <= out_b * 1.001 + np.abs(ref.out) * 2e-7)
    dW = torch.empty((N, K), device="cuda")
    srq.qlinear_bwd_weight(dY, A, qdy, qa, dW, None, ws)
    assert srq.srq_poll_status(ws) == 0
    ref = oracle.qlinear_bwd_weight_e4m3(f(dY), f(A), _oq(qdy), _oq(qa))
    _, out_b = _bound(ref.codes_a, ref.codes_b, ref.scale_a, ref.scale_b)
    assert np.all(np.abs(dW.cpu().numpy().astype(np.float64) - ref.out) <= out_b * 1.001 + np.abs(ref.out) * 2e-7)


def test_floating_point_grid_rejects_other_widths():
    x = synth.normal((64, 64), 1.0, seed=1, device="cuda")
    c = torch.empty((64, 64), dtype=torch.int8, device="cuda")
    sc = torch.empty(1, device="cuda")
    with pytest.raises(srq.SrqError) as e:
        srq.sr_quantize(x, _q(srq.PER_TENSOR, srq.SR, bits=4), c, sc, None, None)
    assert e.value.status == 2
