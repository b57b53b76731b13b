"""Output options of the products against the oracle: accumulation into the output (one binary32
addition per element), re-quantization of the result in the epilogue with a caller-supplied step
(codes bit for bit, saturation included) and the absmax of the result."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import synth

pytestmark = pytest.mark.gpu


def _codes(rows, kc, seed):
    g = torch.Generator().manual_seed(seed)
    full = torch.randint(-127, 128, (rows, (kc + 15) // 16 * 16), generator=g, dtype=torch.int8)
    return full.cuda()[:, :kc]


@pytest.mark.parametrize("M,N,Kc,off", [(300, 520, 256, 0), (129, 257, 130, 5), (64, 256, 4096, 2 ** 34), (520, 96, 384, 8)])
@pytest.mark.parametrize("rnd", [srq.SR, srq.RTN])
@pytest.mark.parametrize("with_out", [True, False])
def test_requantized_output_and_absmax(M, N, Kc, off, rnd, with_out):
    a, b = _codes(M, Kc, 1), _codes(N, Kc, 2)
    s_row = (torch.rand(M) * 0.02 + 1e-3).cuda()
    s_col = (torch.rand(N) * 0.02 + 1e-3).cuda()
    ref_out = oracle.dequant(oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy()), s_row.cpu().numpy(), s_col.cpu().numpy())
    # a step that makes a few percent of the results saturate
    step = torch.tensor([float(np.quantile(np.abs(ref_out), 0.97)) / 127.0], device="cuda")
    q = srq.QSpec(8, srq.PER_TENSOR, rnd, seed=7, tensor_id=11, index_offset=off)
    pad = 16 - N % 16 if N % 16 else 0
    codes_full = torch.full((M, N + pad), 99, dtype=torch.int8, device="cuda")
    codes = codes_full[:, :N]
    absmax = torch.zeros(1, device="cuda")
    out = torch.full((M, N), float("nan"), device="cuda") if with_out else None
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    srq.srq_gemm_i8_ex(a, b, s_row, s_col, out, srq.Output(q=q, step=step, codes=codes, absmax=absmax), None, ws)
    assert srq.srq_poll_status(ws) == 0
    ref_codes, ref_m = oracle.requantize(ref_out, float(step.item()), oracle.QSpec(8, 0, rnd, 7, 11, off))
    got = codes.cpu().numpy()
    bad = np.argwhere(got != ref_codes)
    assert bad.size == 0, f"{len(bad)} code mismatches, first at {bad[0]}: gpu {got[tuple(bad[0])]} oracle {ref_codes[tuple(bad[0])]}"
    assert (np.abs(ref_codes) == 127).mean() > 0.01            # saturation was exercised
    assert absmax.item() == ref_m
    if pad:
        assert bool((codes_full[:, N:] == 99).all())
    if with_out:
        assert np.array_equal(out.cpu().numpy(), ref_out)


@pytest.mark.parametrize("shape", [(264, 392, 328), (512, 256, 4096)])
def test_gradient_accumulation_over_micro_batches(shape):
    """dW += Q(dY)^T Q(A) over three micro-batches equals the oracle's running binary32 sum; small
    outputs with a long contraction take the split path, whose finishing pass accumulates too."""
    T, N, K = shape
    dev = "cuda"
    dW = torch.zeros((N, K), device=dev)
    dA = torch.empty((T, K), device=dev)
    ref = np.zeros((N, K), dtype=np.float32)
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    W = synth.normal((N, K), 0.02, 99, device=dev)
    for mb in range(3):
        A, _, dY = synth.layer_inputs(T, N, K, seed=10 + mb, device=dev, std_dy=1e-3)
        qdy, qa, qw = (srq.QSpec(8, srq.PER_TENSOR, srq.SR, mb, i) for i in (4, 2, 3))
        srq.qlinear_bwd_ex(dY, A, W, qdy, qa, qw, dA, dW, None, srq.Output(accumulate=True), ws)
        assert srq.srq_poll_status(ws) == 0
        r = oracle.qlinear_bwd_weight(dY.cpu().numpy(), A.cpu().numpy(), oracle.QSpec(8, 0, 0, mb, 4), oracle.QSpec(8, 0, 0, mb, 2))
        ref = oracle.accumulate(ref, r.out)
        assert np.array_equal(dW.cpu().numpy(), ref), f"micro-batch {mb}"


def test_layer_chain_without_reading_the_activations_again():
    """Two forward layers: the first writes Q(Y1) for the second in its epilogue (step from the absmax
    of an earlier step, here of a first run); the second layer's product on those codes equals the
    oracle's product on the oracle's re-quantized codes."""
    T, K, N1, N2 = 264, 328, 392, 136
    A, W1, _ = synth.layer_inputs(T, N1, K, seed=3, device="cuda")
    W2 = synth.normal((N2, N1), 0.02, 5, device="cuda")
    qa, qw1, qw2 = srq.QSpec(8, 0, 0, 1, 0), srq.QSpec(8, 0, 0, 1, 1), srq.QSpec(8, 0, 0, 1, 3)
    qy = srq.QSpec(8, 0, srq.SR, 1, 2)
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, max(N1, N2), max(K, N1)))
    # run 1 finds the absmax of Y1 (no fp32 output needed for that either, but it is checked below)
    Y1 = torch.empty((T, N1), device="cuda")
    m = torch.zeros(1, device="cuda")
    srq.qlinear_fwd_ex(A, W1, qa, qw1, Y1, srq.Output(absmax=m), None, ws)
    ref1 = oracle.qlinear_fwd(A.cpu().numpy(), W1.cpu().numpy(), oracle.QSpec(8, 0, 0, 1, 0), oracle.QSpec(8, 0, 0, 1, 1))
    assert m.item() == np.abs(ref1.out).max() and np.array_equal(Y1.cpu().numpy(), ref1.out)
    step = m / 127.0
    # run 2 writes only the codes of Y1
    cy = torch.empty((T, 400), dtype=torch.int8, device="cuda")[:, :N1]      # row pitch a multiple of 16 for the product
    srq.qlinear_fwd_ex(A, W1, qa, qw1, None, srq.Output(q=qy, step=step, codes=cy), None, ws)
    assert srq.srq_poll_status(ws) == 0
    ref_cy, _ = oracle.requantize(ref1.out, float(step.item()), oracle.QSpec(8, 0, 0, 1, 2))
    assert np.array_equal(cy.cpu().numpy(), ref_cy)
    # second layer on those codes
    cw2 = torch.empty((N2, 400), dtype=torch.int8, device="cuda")[:, :N1]
    sw2 = torch.empty(1, device="cuda")
    srq.sr_quantize(W2, qw2, cw2, sw2)
    Y2 = torch.empty((T, N2), device="cuda")
    srq.srq_gemm_i8(cy, cw2, step, sw2, Y2)
    ocw2, osw2, _, _ = oracle.sr_quantize(W2.cpu().numpy(), oracle.QSpec(8, 0, 0, 1, 3))
    ref2 = oracle.dequant(oracle.gemm_i8_nt(ref_cy, ocw2), step.cpu().numpy(), osw2)
    assert np.array_equal(Y2.cpu().numpy(), ref2)


def test_option_errors_are_found_on_the_host():
    a, b = _codes(64, 64, 1), _codes(64, 64, 2)
    one = torch.ones(1, device="cuda")
    with pytest.raises(srq.SrqError):           # neither an output nor codes
        srq.srq_gemm_i8_ex(a, b, one, one, None, srq.Output())
    with pytest.raises(srq.SrqError):           # codes without a step
        srq.srq_gemm_i8_ex(a, b, one, one, None, srq.Output(q=srq.QSpec(8), codes=torch.empty((64, 64), dtype=torch.int8, device="cuda")))
    with pytest.raises(srq.SrqError):           # accumulate without an output
        srq.srq_gemm_i8_ex(a, b, one, one, None, srq.Output(accumulate=True, q=srq.QSpec(8), step=one,
                                                            codes=torch.empty((64, 64), dtype=torch.int8, device="cuda")))


def _bits(t):
    return t.view(torch.uint16).cpu().numpy()


@pytest.mark.parametrize("M,N,Kc", [(300, 520, 256), (129, 257, 130), (64, 256, 4096), (512, 256, 8192), (1, 1, 1), (520, 96, 384)])
@pytest.mark.parametrize("raw_sums", [False, True])
def test_bfloat16_output_is_the_rounded_binary32_result(M, N, Kc, raw_sums):
    """Whole blocks (TMA stores of 32 x 64 boxes), the element-wise path (raw sums requested), the
    split contraction's finishing pass and ragged edges: every stored bfloat16 is the oracle's
    rounding of the oracle's binary32 result, and the pad columns of the buffer stay untouched."""
    a, b = _codes(M, Kc, 1), _codes(N, Kc, 2)
    s_row = (torch.rand(M) * 0.02 + 1e-3).cuda()
    s_col = (torch.rand(N) * 0.02 + 1e-3).cuda()
    acc_ref = oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy())
    ref = oracle.to_bf16(oracle.dequant(acc_ref, s_row.cpu().numpy(), s_col.cpu().numpy()))
    pad = 8 - N % 8 if N % 8 else 0
    full = torch.full((M, N + pad), 7.0, dtype=torch.bfloat16, device="cuda")
    out = full[:, :N]
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda") if raw_sums else None
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    srq.srq_gemm_i8_ex(a, b, s_row, s_col, out, None, acc, ws)
    assert srq.srq_poll_status(ws) == 0
    assert np.array_equal(_bits(out.contiguous()), ref)
    if pad:
        assert bool((full[:, N:] == 7.0).all())
    if raw_sums:
        assert np.array_equal(acc.cpu().numpy(), acc_ref)


def test_bfloat16_output_on_an_unaligned_buffer():
    M, N, Kc = 70, 45, 64
    a, b = _codes(M, Kc, 3), _codes(N, Kc, 4)
    s = torch.tensor([0.01], device="cuda")
    ref = oracle.to_bf16(oracle.dequant(oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy()), np.float32([0.01]), np.float32([0.01])))
    flat = torch.zeros(M * N + 1, dtype=torch.bfloat16, device="cuda")
    out = flat[1:].view(M, N)                      # 2-byte aligned only, odd pitch
    srq.srq_gemm_i8_ex(a, b, s, s, out)
    assert np.array_equal(_bits(out.contiguous()), ref)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_layer_passes_with_bfloat16_outputs_and_fused_codes(dtype):
    """Forward and backward with bfloat16 Y, dA, dW; the codes and the absmax requested next to a
    bfloat16 output still come from the binary32 result."""
    T, N, K = 264, 392, 328
    A, W, dY = synth.layer_inputs(T, N, K, seed=4, dtype=dtype, device="cuda", std_dy=1e-3)
    f = lambda t: t.float().cpu().numpy()
    qs = [srq.QSpec(8, srq.PER_ROW, srq.SR, 9, i) for i in range(5)]
    oq = [oracle.QSpec(8, oracle.PER_ROW, oracle.SR, 9, i) for i in range(5)]
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    r_f = oracle.qlinear_fwd(f(A), f(W), oq[0], oq[1])
    step = torch.tensor([float(np.abs(r_f.out).max()) / 127.0], device="cuda")
    qn = srq.QSpec(8, srq.PER_TENSOR, srq.SR, 9, 20)
    codes = torch.empty((T, 400), dtype=torch.int8, device="cuda")[:, :N]
    m = torch.zeros(1, device="cuda")
    Y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    srq.qlinear_fwd_ex(A, W, qs[0], qs[1], Y, srq.Output(q=qn, step=step, codes=codes, absmax=m), None, ws)
    assert srq.srq_poll_status(ws) == 0
    assert np.array_equal(_bits(Y), oracle.to_bf16(r_f.out))
    rc, rm = oracle.requantize(r_f.out, float(step.item()), oracle.QSpec(8, 0, oracle.SR, 9, 20))
    assert np.array_equal(codes.cpu().numpy(), rc) and m.item() == rm
    dA = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    srq.qlinear_bwd_ex(dY, A, W, qs[4], qs[2], qs[3], dA, dW, None, None, ws)
    assert srq.srq_poll_status(ws) == 0
    assert np.array_equal(_bits(dA), oracle.to_bf16(oracle.qlinear_bwd_input(f(dY), f(W), oq[4], oq[3]).out))
    assert np.array_equal(_bits(dW), oracle.to_bf16(oracle.qlinear_bwd_weight(f(dY), f(A), oq[4], oq[2]).out))


def test_bfloat16_output_cannot_accumulate():
    a, b = _codes(64, 64, 1), _codes(64, 64, 2)
    s = torch.tensor([0.01], device="cuda")
    out = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(srq.SrqError) as e:
        srq.srq_gemm_i8_ex(a, b, s, s, out, srq.Output(accumulate=True))
    assert e.value.status == 2


@pytest.mark.parametrize("M,N,Kc", [(300, 520, 384), (64, 256, 4096)])
def test_int32_accumulation_over_micro_batches_equals_the_product_over_all_of_them(M, N, Kc):
    """accumulate = 2: the raw sums of three micro-batches are added in int32 and the output is formed
    from the total, which is the product over the concatenated contraction, exactly (same step
    sizes for every micro-batch).  The second shape runs the split contraction, whose finishing
    pass does the adding.  A total that does not fit int32 is reported."""
    parts_a = [_codes(M, Kc, 10 + i) for i in range(3)]
    parts_b = [_codes(N, Kc, 20 + i) for i in range(3)]
    s_row = (torch.rand(M) * 0.02 + 1e-3).cuda()
    s_col = (torch.rand(1) * 0.02 + 1e-3).cuda()
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    out = torch.full((M, N), float("nan"), device="cuda")
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    for a, b in zip(parts_a, parts_b):
        srq.srq_gemm_i8_ex(a, b, s_row, s_col, out, srq.Output(accumulate=2), acc, ws)
        assert srq.srq_poll_status(ws) == 0
    ref_acc = oracle.gemm_i8_nt(np.concatenate([a.cpu().numpy() for a in parts_a], 1), np.concatenate([b.cpu().numpy() for b in parts_b], 1))
    assert np.array_equal(acc.cpu().numpy(), ref_acc)
    assert np.array_equal(out.cpu().numpy(), oracle.dequant(ref_acc, s_row.cpu().numpy(), s_col.cpu().numpy()))
    # running sums need their matrix
    with pytest.raises(srq.SrqError) as e:
        srq.srq_gemm_i8_ex(parts_a[0], parts_b[0], s_row, s_col, out, srq.Output(accumulate=2), None, ws)
    assert e.value.status == 1
    # a total beyond int32 wraps and is reported
    acc.fill_(2 ** 31 - 5)
    ones_a = torch.ones((M, 16), dtype=torch.int8, device="cuda")
    ones_b = torch.ones((N, 16), dtype=torch.int8, device="cuda")
    srq.srq_gemm_i8_ex(ones_a, ones_b, s_row, s_col, out, srq.Output(accumulate=2), acc, ws)
    assert srq.srq_poll_status(ws) == 4


def test_layer_weight_gradient_accumulated_in_int32():
    """qlinear_bwd_ex with accumulate = 2 for dW and shared step sizes (srq_qspec_t.absmax of the
    whole batch): two micro-batches give the int32 sums, and dW, of one pass over all tokens."""
    T, N, K = 264, 136, 200
    A, W, dY = synth.layer_inputs(T, N, K, seed=8, device="cuda", std_dy=1e-3)
    mA, mdY = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    srq.srq_absmax(A, mA)
    srq.srq_absmax(dY, mdY)
    f = lambda t: t.cpu().numpy()
    ref = oracle.qlinear_bwd_weight(f(dY), f(A), oracle.QSpec(8, 0, 0, 2, 4), oracle.QSpec(8, 0, 0, 2, 2))
    acc = torch.zeros((N, K), dtype=torch.int32, device="cuda")
    dW = torch.empty((N, K), device="cuda")
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    for lo, hi in ((0, 128), (128, T)):
        qdy = srq.QSpec(8, 0, 0, 2, 4, index_offset=lo * N, absmax=mdY)
        qa = srq.QSpec(8, 0, 0, 2, 2, index_offset=lo * K, absmax=mA)
        dbg = srq.DebugOut(None, None, None, None, acc)
        dA = torch.empty((hi - lo, K), device="cuda")
        srq.qlinear_bwd_ex(dY[lo:hi].contiguous(), A[lo:hi].contiguous(), W, qdy, qa, srq.QSpec(8, 0, 0, 2, 3), dA, dW,
                           None, srq.Output(accumulate=2), ws, dbg_weight=dbg)
        assert srq.srq_poll_status(ws) == 0
    assert np.array_equal(acc.cpu().numpy(), ref.acc)
    assert np.array_equal(dW.cpu().numpy(), ref.out)
