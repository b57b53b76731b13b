"""GPU parity of sr_quantize against the CPU oracle: codes and step sizes bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import synth

pytestmark = pytest.mark.gpu


def _run_gpu(x, q, want_rm=True, want_tr=True, pad_rm=0, pad_tr=0):
    rows, cols = x.shape
    per_row = q.scale == srq.PER_ROW
    dev = x.device
    crm = srm = ctr = strr = None
    if want_rm:
        crm_full = torch.full((rows, cols + pad_rm), 99, dtype=torch.int8, device=dev)
        crm = crm_full[:, :cols]
        srm = torch.full((rows if per_row else 1,), -1.0, dtype=torch.float32, device=dev)
    if want_tr:
        ctr_full = torch.full((cols, rows + pad_tr), 99, dtype=torch.int8, device=dev)
        ctr = ctr_full[:, :rows]
        strr = torch.full((cols if per_row else 1,), -1.0, dtype=torch.float32, device=dev)
    ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(rows, cols), dev)
    srq.sr_quantize(x, q, crm, srm, ctr, strr, ws)
    assert srq.srq_poll_status(ws) == 0
    if want_rm and pad_rm:
        assert bool((crm_full[:, cols:] == 99).all()), "padding of the row-major layout was written"
    if want_tr and pad_tr:
        assert bool((ctr_full[:, rows:] == 99).all()), "padding of the transposed layout was written"
    f = lambda t: None if t is None else t.cpu().numpy()
    return f(crm), f(srm), f(ctr), f(strr)


def _check(x, bits, scale, rnd, seed=0, tid=0, off=0, want_rm=True, want_tr=True, pad_rm=0, pad_tr=0):
    q = srq.QSpec(bits, scale, rnd, seed, tid, off)
    got = _run_gpu(x, q, want_rm, want_tr, pad_rm, pad_tr)
    ref = oracle.sr_quantize(x.float().cpu().numpy(), oracle.QSpec(bits, scale, rnd, seed, tid, off),
                             want_rm, want_tr)
    for name, g, r in zip(("codes_rm", "scale_rm", "codes_tr", "scale_tr"), got, ref):
        if r is None:
            continue
        assert g.shape == r.shape, name
        bad = np.argwhere(g != r)
        assert bad.size == 0, f"{name}: {len(bad)} mismatches, first at {bad[0]}: gpu {g[tuple(bad[0])]} oracle {r[tuple(bad[0])]}"


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
@pytest.mark.parametrize("rnd", [srq.SR, srq.RTN])
@pytest.mark.parametrize("bits", [8, 6, 4, 3])
def test_multi_tile_with_ragged_tail(dtype, scale, rnd, bits):
    # 2.x tiles of 128 in each direction, extents multiples of 4 (vector path)
    x = synth.with_outliers((300, 388), seed=bits, dtype=dtype, device="cuda")
    _check(x, bits, scale, rnd, seed=bits, tid=7, pad_rm=12, pad_tr=4)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shape,off", [((131, 259), 0), ((17, 5), 3), ((1, 1), 0), ((1, 1000), 1),
                                       ((1000, 1), 2), ((129, 130), 2 ** 33 + 2), ((64, 256), 2 ** 40)])
def test_unaligned_extents_and_offsets(dtype, shape, off):
    x = synth.normal(shape, 1.0, seed=shape[0], dtype=dtype, device="cuda")
    for scale in (srq.PER_TENSOR, srq.PER_ROW):
        _check(x, 8, scale, srq.SR, seed=2 ** 40 + 3, tid=2 ** 35 + 1, off=off)
        _check(x, 5, scale, srq.RTN)


def test_single_layout_requests():
    x = synth.normal((200, 136), 1.0, seed=1, device="cuda")
    for scale in (srq.PER_TENSOR, srq.PER_ROW):
        _check(x, 8, scale, srq.SR, want_rm=True, want_tr=False)
        _check(x, 8, scale, srq.SR, want_rm=False, want_tr=True)


def test_strided_input_view():
    big = synth.normal((150, 512), 1.0, seed=2, device="cuda")
    _check(big[:, 64:64 + 260], 8, srq.PER_ROW, srq.SR, seed=1)      # pitch 512, 16-byte aligned start
    _check(big[:, 4:4 + 201], 8, srq.PER_TENSOR, srq.SR, seed=1)      # ragged width, aligned start


def test_zero_tensor_zero_rows_and_tiny_groups():
    z = torch.zeros((130, 132), device="cuda")
    _check(z, 8, srq.PER_TENSOR, srq.SR)
    x = synth.normal((130, 132), 1.0, seed=3, device="cuda")
    x[5] = 0
    x[:, 9] = 0
    x[7] = 1e-39          # reciprocal step overflows: the group is flushed to zero
    _check(x, 8, srq.PER_ROW, srq.SR)
    _check(x, 4, srq.PER_ROW, srq.RTN)


def test_grid_exact_inputs_and_extreme_element():
    k = torch.arange(-127, 128, dtype=torch.float32, device="cuda").repeat(4, 1) * 2.0 ** -5
    for seed in range(3):
        _check(k.contiguous(), 8, srq.PER_TENSOR, srq.SR, seed=seed)
    c = torch.empty((4, 255), dtype=torch.int8, device="cuda")
    s = torch.empty(1, device="cuda")
    srq.sr_quantize(k.contiguous(), srq.QSpec(seed=5), c, s)
    assert torch.equal(c.float(), k * 32)


def test_same_spec_same_codes_other_spec_other_codes():
    x = synth.normal((256, 256), 1.0, seed=4, device="cuda")
    a = _run_gpu(x, srq.QSpec(8, 0, 0, 1, 2))[0]
    b = _run_gpu(x, srq.QSpec(8, 0, 0, 1, 2))[0]
    c = _run_gpu(x, srq.QSpec(8, 0, 0, 1, 3))[0]
    d = _run_gpu(x, srq.QSpec(8, 0, 0, 2, 2))[0]
    assert np.array_equal(a, b)
    assert (a != c).mean() > 0.2 and (a != d).mean() > 0.2


def test_nonfinite_input_is_reported():
    x = synth.normal((64, 64), 1.0, seed=5, device="cuda")
    x[3, 3] = float("inf")
    ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(64, 64))
    c = torch.empty((64, 64), dtype=torch.int8, device="cuda")
    s = torch.empty(1, device="cuda")
    srq.sr_quantize(x, srq.QSpec(), c, s, ws=ws)
    assert srq.srq_poll_status(ws) == 6
    x[3, 3] = float("nan")
    srq.sr_quantize(x, srq.QSpec(scale=srq.PER_ROW), c, torch.empty(64, device="cuda"), ws=ws)
    assert srq.srq_poll_status(ws) == 6
    x[3, 3] = 1.0
    srq.sr_quantize(x, srq.QSpec(), c, s, ws=ws)
    assert srq.srq_poll_status(ws) == 0


def test_unbiasedness_of_1e4_draws_on_the_gpu():
    """E[Q(x)] = x within 5 sigma and Var <= D^2/4, 4096-element tensor, 10^4 seeds."""
    x = synth.normal((1, 4096), 1.0, seed=6, device="cuda")
    draws = 10_000
    c = torch.empty((1, 4096), dtype=torch.int8, device="cuda")
    s = torch.empty(1, device="cuda")
    ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(1, 4096))
    acc = torch.zeros((1, 4096), dtype=torch.float64, device="cuda")
    acc2 = torch.zeros_like(acc)
    for seed in range(draws):
        srq.sr_quantize(x, srq.QSpec(8, 0, 0, seed, 3), c, s, ws=ws)
        acc += c
        acc2 += c.double() ** 2
    xs = x.cpu().numpy()
    d, inv = oracle.scale_from_absmax(float(np.abs(xs).max()), 8)
    assert s.item() == d
    t = xs.astype(np.float64) * float(inv)
    p = t - np.floor(t)
    mean = (acc / draws).cpu().numpy()
    var = (acc2 / draws).cpu().numpy() - mean ** 2
    assert np.all(np.abs(mean - t) <= 5 * np.sqrt(p * (1 - p) / draws) + 3.0 / draws)
    assert var.max() <= 0.25 + 1e-9
    # the first few draws agree with the oracle exactly (same generator, same rule)
    for seed in (0, 1, 9999):
        srq.sr_quantize(x, srq.QSpec(8, 0, 0, seed, 3), c, s, ws=ws)
        ref = oracle.sr_quantize(xs, oracle.QSpec(8, 0, 0, seed, 3))[0]
        assert np.array_equal(c.cpu().numpy(), ref)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_absmax_entry_point_and_a_known_absmax(dtype):
    """srq_absmax equals the plain maximum; a quantization point that carries it skips its own
    absmax pass and gives the same codes and step size (also a larger, all-reduced-like maximum
    works: then the oracle is given a tensor whose maximum is that value)."""
    x = synth.with_outliers((300, 388), seed=8, dtype=dtype, device="cuda")
    m = torch.full((1,), -1.0, device="cuda")
    srq.srq_absmax(x, m)
    assert m.item() == x.float().abs().max().item()
    srq.srq_absmax(x[:, 8:209], m)                       # strided view (16-byte aligned start), ragged width
    assert m.item() == x[:, 8:209].float().abs().max().item()
    srq.srq_absmax(x, m)
    for rnd in (srq.SR, srq.RTN):
        a = _run_gpu(x, srq.QSpec(8, srq.PER_TENSOR, rnd, 3, 4))
        b = _run_gpu(x, srq.QSpec(8, srq.PER_TENSOR, rnd, 3, 4, absmax=m))
        for g, r in zip(a, b):
            assert np.array_equal(g, r)
    # a maximum larger than this tensor's own (as after a maximum over several shards)
    big = torch.tensor([m.item() * 1.7], device="cuda")
    got = _run_gpu(x, srq.QSpec(6, srq.PER_TENSOR, srq.SR, 3, 4, absmax=big))
    xs = torch.cat([x.float().cpu(), torch.tensor([[big.item()] + [0.0] * 387])], 0).numpy()   # same maximum for the oracle
    ref = oracle.sr_quantize(xs, oracle.QSpec(6, 0, 0, 3, 4), True, True)
    assert np.array_equal(got[0], ref[0][:300]) and np.array_equal(got[1], ref[1])
    assert np.array_equal(got[2], ref[2][:, :300])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
def test_eight_random_bits_per_element(dtype, scale):
    """SRQ_SR8 against the oracle: aligned tiles (one Philox block per 16 elements, shared by four lanes),
    ragged shapes and index offsets that break the 16-element alignment (element-wise path)."""
    x = synth.with_outliers((300, 400), seed=12, dtype=dtype, device="cuda")
    _check(x, 8, scale, srq.SR8, seed=7, tid=3, off=0)
    _check(x, 4, scale, srq.SR8, seed=7, tid=3, off=2 ** 36 + 32)
    _check(x, 8, scale, srq.SR8, seed=1, tid=2, off=8)                 # offset not a multiple of 16
    _check(x[:, :388].contiguous(), 6, scale, srq.SR8, seed=2)          # width not a multiple of 16
    y = synth.normal((131, 259), 1.0, seed=5, dtype=dtype, device="cuda")
    _check(y, 8, scale, srq.SR8, seed=3, off=5)
    _check(x, 8, scale, srq.SR8, want_rm=False, want_tr=True)
    with pytest.raises(srq.SrqError):                                    # integer grid only
        srq.sr_quantize(x, srq.QSpec(8, scale, srq.SR8, format=srq.GRID_E4M3),
                        torch.empty((300, 400), dtype=torch.int8, device="cuda"), torch.empty(300, device="cuda"))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shape,off", [((70, 512), 0), ((33, 4096), 4), ((5, 8192), 2 ** 34), ((130, 2052), 8),
                                       ((2000, 516), 0), ((3, 8196), 0)])
def test_one_pass_per_row_path_matches_the_oracle(dtype, shape, off):
    """Per-row steps with row-major codes only: rows of 512 .. 8192 elements take the kernel that
    reads the input once (row maximum and codes from the same registers); more rows than resident
    CTAs, partly filled groups per thread, a zero row, a row too small to scale, padded code
    pitch.  The 8196-column case is past its limit and takes the two-pass path: same codes."""
    x = synth.with_outliers(shape, seed=shape[1], dtype=dtype, device="cuda")
    x[0] = 0
    x[shape[0] - 1] = 1e-39 if dtype == torch.float32 else 0.0
    for bits, rnd in ((8, srq.SR), (4, srq.SR), (6, srq.RTN)):
        _check(x, bits, srq.PER_ROW, rnd, seed=11, tid=2 ** 33 + 5, off=off, want_rm=True, want_tr=False, pad_rm=12)
    # the same rows through the two-pass kernels (both layouts requested) give the same row-major codes
    q = srq.QSpec(8, srq.PER_ROW, srq.SR, 11, 3, off)
    one = _run_gpu(x, q, True, False)
    two = _run_gpu(x, q, True, True)
    assert np.array_equal(one[0], two[0]) and np.array_equal(one[1], two[1])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shape", [(300, 388), (262, 131)])
def test_token_shards_with_per_row_steps_share_their_column_maxima(dtype, shape):
    """Per-row mode, transposed layout: its groups are the columns of the source, which run over the
    tokens.  Two token shards that exchange their column maxima (srq_absmax_cols, then an element-wise
    maximum as an all-reduce would form it) produce exactly the columns of codes, and the step sizes,
    that one device produces on the whole tensor; row-major codes need no exchange."""
    rows, cols = shape
    x = synth.with_outliers(shape, seed=21, dtype=dtype, device="cuda")
    x[:, 3] = 0
    cut = 136
    shards = [x[:cut].contiguous(), x[cut:].contiguous()]
    cm = [torch.full((cols,), -1.0, device="cuda") for _ in shards]
    for sh, m in zip(shards, cm):
        srq.srq_absmax_cols(sh, m)
        assert torch.equal(m, sh.float().abs().amax(dim=0))
    shared = torch.maximum(cm[0], cm[1])
    for bits, rnd in ((8, srq.SR), (4, srq.RTN)):
        whole = oracle.sr_quantize(x.float().cpu().numpy(), oracle.QSpec(bits, oracle.PER_ROW, rnd, 5, 9), True, True)
        first = 0
        for sh in shards:
            q = srq.QSpec(bits, srq.PER_ROW, rnd, 5, 9, index_offset=first * cols, absmax=shared)
            for want_rm in (True, False):
                got = _run_gpu(sh, q, want_rm, True)
                n = sh.shape[0]
                assert np.array_equal(got[2], whole[2][:, first:first + n]), "transposed codes of the shard"
                assert np.array_equal(got[3], whole[3]), "column step sizes"
                if want_rm:
                    assert np.array_equal(got[0], whole[0][first:first + n]) and np.array_equal(got[1], whole[1][first:first + n])
            first += sh.shape[0]
    # the weight-gradient product of the shards then adds up to the unsharded one, int32 sums exactly
    A = synth.normal((rows, 72), 1.0, seed=3, dtype=dtype, device="cuda")
    ma, mx = torch.empty(72, device="cuda"), torch.empty(cols, device="cuda")
    srq.srq_absmax_cols(A, ma)
    srq.srq_absmax_cols(x, mx)
    f = lambda t: t.float().cpu().numpy()
    ref = oracle.qlinear_bwd_weight(f(x), f(A), oracle.QSpec(8, oracle.PER_ROW, oracle.SR, 1, 4), oracle.QSpec(8, oracle.PER_ROW, oracle.SR, 1, 2))
    total = np.zeros_like(ref.acc, dtype=np.int64)
    first = 0
    for lo, hi in ((0, cut), (cut, rows)):
        T = hi - lo
        dW = torch.empty((cols, 72), device="cuda")
        acc = torch.empty((cols, 72), dtype=torch.int32, device="cuda")
        dbg = srq.DebugOut(None, torch.empty(cols, device="cuda"), None, torch.empty(72, device="cuda"), acc)
        srq.qlinear_bwd_weight(x[lo:hi].contiguous(), A[lo:hi].contiguous(),
                               srq.QSpec(8, srq.PER_ROW, srq.SR, 1, 4, index_offset=lo * cols, absmax=mx),
                               srq.QSpec(8, srq.PER_ROW, srq.SR, 1, 2, index_offset=lo * 72, absmax=ma), dW, dbg)
        assert np.array_equal(dbg.scale_a.cpu().numpy(), ref.scale_a) and np.array_equal(dbg.scale_b.cpu().numpy(), ref.scale_b)
        total += acc.cpu().numpy()
    assert np.array_equal(total, ref.acc.astype(np.int64))


def test_one_pass_per_row_path_reports_nonfinite_input():
    x = synth.normal((40, 1024), 1.0, seed=5, device="cuda")
    x[7, 900] = float("nan")
    ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(40, 1024))
    c = torch.empty((40, 1024), dtype=torch.int8, device="cuda")
    s = torch.empty(40, device="cuda")
    srq.sr_quantize(x, srq.QSpec(scale=srq.PER_ROW), c, s, ws=ws)
    assert srq.srq_poll_status(ws) == 6
    x[7, 900] = float("-inf")
    srq.sr_quantize(x, srq.QSpec(scale=srq.PER_ROW, round=srq.RTN), c, s, ws=ws)
    assert srq.srq_poll_status(ws) == 6
    x[7, 900] = 0.5
    srq.sr_quantize(x, srq.QSpec(scale=srq.PER_ROW), c, s, ws=ws)
    assert srq.srq_poll_status(ws) == 0


@pytest.mark.parametrize("case", range(32))
def test_random_shapes_pitches_offsets_and_modes(case):
    """Seeded random cases over extents (ragged and aligned, rows long enough for the one-pass per-row
    kernel included), input pitches, index offsets, widths, grids of modes and layouts."""
    rng = np.random.default_rng(1000 + case)
    rows = int(rng.integers(1, 260))
    cols = int(rng.choice([rng.integers(1, 200), rng.integers(500, 1200), 4 * rng.integers(128, 300), 1024, 2048]))
    ld = cols + int(rng.choice([0, 0, 4, 8, 3]))
    dtype = [torch.float32, torch.bfloat16][int(rng.integers(2))]
    scale = [srq.PER_TENSOR, srq.PER_ROW][int(rng.integers(2))]
    rnd = [srq.SR, srq.RTN, srq.SR8][int(rng.integers(3))]
    bits = int(rng.integers(2, 9))
    off = int(rng.choice([0, 4, 16, 5, 2 ** 32 - 8, 2 ** 35 + 12]))
    want_rm, want_tr = [(True, True), (True, False), (False, True)][int(rng.integers(3))]
    base = synth.with_outliers((rows, ld), seed=case, dtype=dtype, device="cuda")
    x = base[:, :cols]
    if case % 5 == 0:
        x[rows // 2] = 0
    q = srq.QSpec(bits, scale, rnd, seed=case, tensor_id=2 ** 32 + case, index_offset=off)
    got = _run_gpu(x, q, want_rm, want_tr, pad_rm=int(rng.choice([0, 4, 7])), pad_tr=int(rng.choice([0, 4, 5])))
    ref = oracle.sr_quantize(x.float().cpu().numpy(), oracle.QSpec(bits, scale, rnd, case, 2 ** 32 + case, off), want_rm, want_tr)
    for name, g, r in zip(("codes_rm", "scale_rm", "codes_tr", "scale_tr"), got, ref):
        if r is None:
            continue
        bad = np.argwhere(g != r)
        assert bad.size == 0, f"{name}: {len(bad)} mismatches, first at {bad[0]} ({rows}x{cols}, ld {ld}, {dtype}, scale {scale}, round {rnd}, bits {bits}, off {off})"
