"""GPU parity of the int8 tensor-core product and its dequantizing epilogue."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq

pytestmark = pytest.mark.gpu


def _codes(rows, kc, seed, lo=-127, hi=127, pad=None):
    g = torch.Generator(device="cpu").manual_seed(seed)
    pitch = (kc + 15) // 16 * 16 if pad is None else pad
    full = torch.zeros((rows, pitch), dtype=torch.int8)
    full[:, :kc] = torch.randint(lo, hi + 1, (rows, kc), generator=g, dtype=torch.int8)
    if pitch > kc:
        full[:, kc:] = 77        # padding must never be read as data
    return full.cuda()[:, :kc]


def _run(a, b, s_row, s_col, want_acc=True):
    M, N = a.shape[0], b.shape[0]
    out = torch.full((M, N), float("nan"), device="cuda")
    acc = torch.full((M, N), -1, dtype=torch.int32, device="cuda") if want_acc else None
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    srq.srq_gemm_i8(a, b, s_row, s_col, out, acc, ws)
    st = srq.srq_poll_status(ws)
    assert st == 0, srq.status_string(st)
    return out.cpu().numpy(), None if acc is None else acc.cpu().numpy()


@pytest.mark.parametrize("M,N,Kc", [(64, 256, 256), (128, 256, 128), (1, 1, 1), (5, 7, 3), (129, 257, 130),
                                    (300, 520, 1000), (128, 512, 4096), (200, 40, 48), (384, 768, 640)])
@pytest.mark.parametrize("per_row", [False, True])
def test_product_and_dequant_match_the_oracle(M, N, Kc, per_row):
    a, b = _codes(M, Kc, 1), _codes(N, Kc, 2)
    g = torch.Generator(device="cpu").manual_seed(3)
    s_row = (torch.rand(M if per_row else 1, generator=g) * 0.1 + 1e-3).cuda()
    s_col = (torch.rand(N if per_row else 1, generator=g) * 0.1 + 1e-3).cuda()
    out, acc = _run(a, b, s_row, s_col)
    ref_acc = oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy())
    assert np.array_equal(acc, ref_acc)
    ref_out = oracle.dequant(ref_acc, s_row.cpu().numpy(), s_col.cpu().numpy())
    assert np.array_equal(out, ref_out)          # same two binary32 multiplies: 0 ulp
    # without the raw sums the results leave through the block-store path: same values
    out2, _ = _run(a, b, s_row, s_col, want_acc=False)
    assert np.array_equal(out2, ref_out)


def test_longest_contraction_with_extreme_codes_fills_int32_without_overflow():
    """Kc = 133136 is the longest 16-aligned contraction the int32 rule admits at 8 bits
    (133136 * 127^2 = 2147350544 < 2^31).  With every code at +-127 each sum is +-that number, on
    the unsplit path (raw sums requested) and on the split path, whose partial sums are added in
    memory: no intermediate may wrap."""
    Kc, M, N = 133136, 130, 260
    top = Kc * 127 * 127
    assert top < 2 ** 31 <= (Kc + 16) * 127 * 127
    sign_a = torch.where(torch.arange(M) % 3 == 0, -1, 1).to(torch.int8)
    sign_b = torch.where(torch.arange(N) % 5 == 0, -1, 1).to(torch.int8)
    a = (sign_a[:, None] * torch.full((M, Kc), 127, dtype=torch.int8)).cuda()
    b = (sign_b[:, None] * torch.full((N, Kc), 127, dtype=torch.int8)).cuda()
    want = (sign_a[:, None].int() * sign_b[None, :].int()).numpy().astype(np.int64) * top
    s_row = torch.full((M,), 2.0 ** -20, device="cuda")
    s_col = torch.full((1,), 3.0, device="cuda")
    ref_out = oracle.dequant(want.astype(np.int32), s_row.cpu().numpy(), s_col.cpu().numpy())
    for want_acc in (True, False):
        out, acc = _run(a, b, s_row, s_col, want_acc=want_acc)
        if want_acc:
            assert np.array_equal(acc.astype(np.int64), want)
        assert np.array_equal(out, ref_out)
    # one more 16-byte step of the contraction is refused before anything is launched
    a2 = torch.zeros((M, Kc + 16), dtype=torch.int8, device="cuda")
    b2 = torch.zeros((N, Kc + 16), dtype=torch.int8, device="cuda")
    with pytest.raises(srq.SrqError) as e:
        srq.srq_gemm_i8(a2, b2, s_row, s_col, torch.empty((M, N), device="cuda"))
    assert e.value.status == 4


def test_special_code_matrices():
    # all ones: every sum equals the contraction length; identity: returns the other operand
    Kc = 400
    ones = torch.ones((130, 400), dtype=torch.int8, device="cuda")
    one = torch.ones(1, device="cuda")
    out, acc = _run(ones[:, :Kc], ones[:70, :Kc], one, one)
    assert (acc == Kc).all() and (out == Kc).all()
    eye = torch.eye(256, dtype=torch.int8, device="cuda")
    b = _codes(300, 256, 5)
    out, acc = _run(eye, b, one, one)
    assert np.array_equal(acc, b.cpu().numpy().T.astype(np.int32))
    # extreme codes over the longest contraction of the workloads: 65536 * 127^2 < 2^31
    a = torch.full((128, 65536), 127, dtype=torch.int8, device="cuda")
    bb = torch.full((256, 65536), -127, dtype=torch.int8, device="cuda")
    out, acc = _run(a, bb, one, one)
    assert (acc == -65536 * 127 * 127).all()


def test_split_contraction_is_exact():
    # small output, long contraction: the kernel splits K across CTAs and adds int32 partials
    for (M, N, Kc) in [(768, 768, 8192), (256, 256, 16384), (100, 300, 4224)]:
        a, b = _codes(M, Kc, 11), _codes(N, Kc, 12)
        s_row = torch.rand(M, device="cuda") + 0.5
        s_col = torch.rand(N, device="cuda") + 0.5
        out, acc = _run(a, b, s_row, s_col)
        ref_acc = oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy())
        assert np.array_equal(acc, ref_acc)
        assert np.array_equal(out, oracle.dequant(ref_acc, s_row.cpu().numpy(), s_col.cpu().numpy()))
        out1, _ = _run(a, b, s_row, s_col, want_acc=False)     # split, partial sums added by block reductions
        assert np.array_equal(out1, out)
        # and without the workspace (unsplit path) the result is the same
        out2 = torch.empty((M, N), device="cuda")
        ws = srq.new_workspace(256)
        srq.srq_gemm_i8(a, b, s_row, s_col, out2, None, ws)
        assert srq.srq_poll_status(ws) == 0
        assert np.array_equal(out2.cpu().numpy(), out)


def test_many_tiles_per_cta_and_freivalds():
    """More tiles than SMs (persistent loop, both TMEM buffers, ring wrap-around), checked
    with exact integer Freivalds products and 64 fully recomputed rows."""
    M, N, Kc = 128 * 40, 256 * 9, 768
    a, b = _codes(M, Kc, 21), _codes(N, Kc, 22)
    one = torch.ones(1, device="cuda")
    out, acc = _run(a, b, one, one)
    rng = np.random.default_rng(0)
    rows = np.sort(rng.choice(M, 64, replace=False))
    ref = oracle.gemm_i8_nt(a.cpu().numpy()[rows], b.cpu().numpy())
    assert np.array_equal(acc[rows], ref)
    A64, B64, C64 = a.cpu().numpy().astype(np.int64), b.cpu().numpy().astype(np.int64), acc.astype(np.int64)
    for _ in range(3):
        r = rng.integers(-3, 4, (N, 1))
        assert np.array_equal(C64 @ r, A64 @ (B64.T @ r))
        l = rng.integers(-3, 4, (1, M))
        assert np.array_equal(l @ C64, (l @ A64) @ B64.T)
    assert np.array_equal(out, acc.astype(np.float32))
    out2, _ = _run(a, b, one, one, want_acc=False)
    assert np.array_equal(out2, out)


@pytest.mark.parametrize("M,N,Kc,pad", [(300, 260, 256, 0), (257, 36, 130, 4), (4096, 96, 512, 0), (520, 1000, 384, 24), (130, 70, 64, 1), (140, 258, 64, 2), (300, 521, 128, 3)])
def test_output_pitch_and_ragged_edges_on_the_block_store_path(M, N, Kc, pad):
    """No raw sums requested: every result goes through shared memory and a clipped block store.
    The output has a row pitch larger than N and guard values around it that must survive."""
    a, b = _codes(M, Kc, 31), _codes(N, Kc, 32)
    s_row = torch.rand(M, device="cuda") + 0.5
    s_col = torch.rand(N, device="cuda") + 0.5
    full = torch.full((M + 2, N + pad + 8), 7.5, device="cuda")
    out = full[1:M + 1, 4:4 + N] if pad else full[1:M + 1, :N]
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    srq.srq_gemm_i8(a, b, s_row, s_col, out, None, ws)
    assert srq.srq_poll_status(ws) == 0
    ref = oracle.dequant(oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy()), s_row.cpu().numpy(), s_col.cpu().numpy())
    assert np.array_equal(out.cpu().numpy(), ref)
    guard = full.clone()
    guard[1:M + 1, (4 if pad else 0):(4 if pad else 0) + N] = 7.5
    assert bool((guard == 7.5).all()), "a store went outside the output"


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_survives():
    """Failure detection without a fault: a wait on a barrier that nothing signals gives up after its
    limit, the status word says so, and the next call on the same context works."""
    import time
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(128, 256))
    t0 = time.perf_counter()
    srq.srq_selftest_bounded_wait(ws, limit_us=2000)
    assert srq.srq_poll_status(ws) == 7
    assert time.perf_counter() - t0 < 1.0
    assert srq.status_string(7) == "bounded wait in a kernel ran out"
    a, b = _codes(128, 256, 1), _codes(256, 256, 2)
    one = torch.ones(1, device="cuda")
    out, acc = _run(a, b, one, one)
    assert np.array_equal(acc, oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy()))


@pytest.mark.parametrize("case", range(24))
def test_random_products(case):
    """Seeded random products: extents from one element to several tiles (one-CTA and CTA-pair
    tiles, split and unsplit contractions), output pitches, per-tensor and per-row step sizes,
    fp32 or bfloat16 results, with and without the raw sums."""
    rng = np.random.default_rng(500 + case)
    M = int(rng.choice([rng.integers(1, 129), rng.integers(129, 700), 256, 512]))
    N = int(rng.choice([rng.integers(1, 300), rng.integers(300, 800), 256, 768]))
    Kc = int(rng.choice([rng.integers(1, 300), 16 * rng.integers(8, 400), 4096]))
    a, b = _codes(M, Kc, 2 * case), _codes(N, Kc, 2 * case + 1)
    per_row = bool(rng.integers(2))
    s_row = (torch.rand(M if per_row else 1) * 0.1 + 1e-3).cuda()
    s_col = (torch.rand(N if per_row else 1) * 0.1 + 1e-3).cuda()
    bf16 = bool(rng.integers(2))
    want_acc = bool(rng.integers(2))
    pad = int(rng.choice([0, 0, 8, 3]))
    full = torch.full((M, N + pad), 7.0, dtype=torch.bfloat16 if bf16 else torch.float32, device="cuda")
    out = full[:, :N]
    acc = torch.full((M, N), -1, dtype=torch.int32, device="cuda") if want_acc else None
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    srq.srq_gemm_i8_ex(a, b, s_row, s_col, out, None, acc, ws)
    assert srq.srq_poll_status(ws) == 0
    ref_acc = oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy())
    ref = oracle.dequant(ref_acc, s_row.cpu().numpy(), s_col.cpu().numpy())
    tag = f"M {M} N {N} Kc {Kc} per_row {per_row} bf16 {bf16} acc {want_acc} pad {pad}"
    if want_acc:
        assert np.array_equal(acc.cpu().numpy(), ref_acc), tag
    if bf16:
        assert np.array_equal(out.contiguous().view(torch.uint16).cpu().numpy(), oracle.to_bf16(ref)), tag
    else:
        assert np.array_equal(out.cpu().numpy(), ref), tag
    if pad:
        assert bool((full[:, N:] == 7.0).all()), tag + ": pad columns written"


def test_tensor_pipe_microbenchmark_runs_and_counts_its_operations():
    """The issue-rate microbenchmark (no global traffic) finishes with a clean status and reports
    2 * 256 * 256 * 128 operations per CTA pair and k-block; odd counts take the short last chunk."""
    ws = srq.new_workspace(256)
    pairs = torch.cuda.get_device_properties(0).multi_processor_count // 2
    for kb in (1, 7, 8, 9, 17, 64, 515):
        ops = srq.srq_selftest_mma_rate(ws, kb)
        assert srq.srq_poll_status(ws) == 0
        assert ops > 0 and ops % (kb * 2 * 256 * 256 * 128) == 0 and ops // (kb * 2 * 256 * 256 * 128) <= pairs
    with pytest.raises(srq.SrqError):
        srq.srq_selftest_mma_rate(ws, 0)


def test_product_timer_brackets_the_launches_and_changes_no_result():
    """srq_set_product_timer: the next launches write their device-side start and end times into the
    caller's slots, in order; launches beyond the slots and launches after it is switched off are not
    timed; results stay those of the untimed call."""
    a, b = _codes(512, 1024, 1), _codes(512, 1024, 2)
    one = torch.ones(1, device="cuda")
    want, _ = _run(a, b, one, one, want_acc=False)
    slots = srq.new_product_timer(2)
    srq.srq_set_product_timer(slots)
    try:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        outs = [_run(a, b, one, one, want_acc=False)[0] for _ in range(3)]      # the third finds no slot
        e1.record()
        torch.cuda.synchronize()
    finally:
        srq.srq_set_product_timer(None)
    t = slots.cpu().numpy()
    dur = t[:, 1] - t[:, 0]
    assert (t[:, 0] > 0).all() and (dur > 0).all() and (dur < e0.elapsed_time(e1) * 1e6).all()
    assert t[1, 0] >= t[0, 1]                                   # the second launch starts after the first has ended
    for o in outs:
        assert np.array_equal(o, want)
    again = srq.new_product_timer(1)
    _run(a, b, one, one, want_acc=False)                        # switched off: nothing is written
    assert again[0, 1].item() == 0
