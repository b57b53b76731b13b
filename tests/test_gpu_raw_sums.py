"""Raw int32 sums as the output of a product, and the finishing step on its own (srq_dequant_i32):
the exact route to the weight gradient of a batch whose tokens sit on several devices.  Integer
sums add exactly in any order, so shards' sums added together and scaled once must give, bit for
bit, what one product over the whole batch gives."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _codes(rows, kc, seed):
    g = torch.Generator().manual_seed(seed)
    full = torch.randint(-127, 128, (rows, (kc + 15) // 16 * 16), generator=g, dtype=torch.int8)
    return full.cuda()[:, :kc]


# block-store path (N % 4 == 0), element-wise path (odd N), split contraction (small output, long Kc)
@pytest.mark.parametrize("M,N,Kc", [(300, 520, 256), (129, 257, 130), (512, 256, 8192), (64, 256, 4096), (1, 1, 1), (384, 768, 2048)])
def test_raw_sums_equal_the_oracles_int32_sums_and_dequant_i32_finishes_them(M, N, Kc):
    a, b = _codes(M, Kc, 1), _codes(N, Kc, 2)
    s_row = (torch.rand(M, generator=torch.Generator().manual_seed(3)) * 0.02 + 1e-3).cuda()
    s_col = (torch.rand(N, generator=torch.Generator().manual_seed(4)) * 0.02 + 1e-3).cuda()
    pad = 3
    sums_full = torch.full((M, N + pad), -7, dtype=torch.int32, device="cuda")
    sums = sums_full[:, :N] if N % 4 else sums_full[:, :N].contiguous()
    ws = srq.new_workspace(srq.srq_gemm_workspace_bytes(M, N))
    srq.srq_gemm_i8_ex(a, b, s_row, s_col, sums, None, None, ws)
    assert srq.srq_poll_status(ws) == 0
    ref_acc = oracle.gemm_i8_nt(a.cpu().numpy(), b.cpu().numpy())
    assert np.array_equal(sums.cpu().numpy(), ref_acc)
    if N % 4:
        assert bool((sums_full[:, N:] == -7).all())            # pad columns untouched
    ref_out = oracle.dequant(ref_acc, s_row.cpu().numpy(), s_col.cpu().numpy())
    out = torch.full((M, N), float("nan"), device="cuda")
    srq.srq_dequant_i32(sums, s_row, s_col, out)
    assert np.array_equal(out.cpu().numpy(), ref_out)
    # per-tensor step sizes, bfloat16 output
    out16 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    srq.srq_dequant_i32(sums, s_row[:1], s_col[:1], out16)
    ref16 = oracle.to_bf16(oracle.dequant(ref_acc, s_row[:1].cpu().numpy(), s_col[:1].cpu().numpy()))
    assert np.array_equal(out16.view(torch.int16).cpu().numpy().view(np.uint16), ref16)


@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
def test_two_token_shards_give_the_unsharded_weight_gradient_bit_for_bit(scale):
    """Two shards of the tokens, run one after the other on this device as two ranks would run them:
    shared maxima (srq_absmax / srq_absmax_cols, max-reduced), index_offset = first_row * cols, raw
    sums of dW added as integers, scaled once.  Compared with the oracle on the whole batch."""
    T, N, K = 640, 264, 392
    per_row = scale == srq.PER_ROW
    A, W, dY = synth.layer_inputs(T, N, K, 5, torch.float32, "cuda", std_dy=1e-3)
    half = T // 2
    ws = srq.new_workspace(srq.srq_workspace_bytes(half, N, K))
    n_a, n_dy = (K, N) if per_row else (1, 1)
    # maxima of each shard, then their element-wise maximum (what an all-reduce(max) leaves on every rank)
    ma, mdy = torch.zeros((2, n_a), device="cuda"), torch.zeros((2, n_dy), device="cuda")
    for r in range(2):
        a, dy = A[r * half:(r + 1) * half], dY[r * half:(r + 1) * half]
        if per_row:
            srq.srq_absmax_cols(a, ma[r]); srq.srq_absmax_cols(dy, mdy[r])
        else:
            srq.srq_absmax(a, ma[r]); srq.srq_absmax(dy, mdy[r])
    ma, mdy = ma.max(dim=0).values.contiguous(), mdy.max(dim=0).values.contiguous()
    total = torch.zeros((N, K), dtype=torch.int32, device="cuda")
    s_dy = torch.empty(N if per_row else 1, device="cuda")
    s_a = torch.empty(K if per_row else 1, device="cuda")
    dA = torch.empty((T, K), device="cuda")
    for r in range(2):
        a, dy = A[r * half:(r + 1) * half], dY[r * half:(r + 1) * half]
        qdy = srq.QSpec(8, scale, srq.SR, 11, 4, r * half * N, absmax=mdy)
        qa = srq.QSpec(8, scale, srq.SR, 11, 2, r * half * K, absmax=ma)
        qw = srq.QSpec(8, scale, srq.SR, 11, 3)
        sums = torch.empty((N, K), dtype=torch.int32, device="cuda")
        srq.qlinear_bwd_ex(dy, a, W, qdy, qa, qw, dA[r * half:(r + 1) * half], sums, None, None, ws,
                           dbg_weight=srq.DebugOut(scale_a=s_dy, scale_b=s_a))
        assert srq.srq_poll_status(ws) == 0
        total += sums                                            # the all-reduce(sum) of the ranks
    dW = torch.empty((N, K), device="cuda")
    srq.srq_dequant_i32(total, s_dy, s_a, dW)
    om = oracle.PER_ROW if per_row else oracle.PER_TENSOR
    full = oracle.qlinear_bwd_weight(dY.cpu().numpy(), A.cpu().numpy(), oracle.QSpec(8, om, oracle.SR, 11, 4),
                                     oracle.QSpec(8, om, oracle.SR, 11, 2))
    assert np.array_equal(total.cpu().numpy(), full.acc)
    assert np.array_equal(s_dy.cpu().numpy(), full.scale_a) and np.array_equal(s_a.cpu().numpy(), full.scale_b)
    assert np.array_equal(dW.cpu().numpy(), full.out)
    if not per_row:       # dA rows need no exchange (per row, dY's token scales are local by construction too)
        full_i = oracle.qlinear_bwd_input(dY.cpu().numpy(), W.cpu().numpy(), oracle.QSpec(8, om, oracle.SR, 11, 4),
                                          oracle.QSpec(8, om, oracle.SR, 11, 3))
        assert np.array_equal(dA.cpu().numpy(), full_i.out)


def test_raw_sums_do_not_combine_with_other_output_options():
    a, b = _codes(64, 64, 1), _codes(64, 64, 2)
    one = torch.ones(1, device="cuda")
    sums = torch.empty((64, 64), dtype=torch.int32, device="cuda")
    for o in (srq.Output(accumulate=1), srq.Output(absmax=torch.zeros(1, device="cuda"))):
        with pytest.raises(srq.SrqError) as e:
            srq.srq_gemm_i8_ex(a, b, one, one, sums, o)
        assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(srq.SrqError) as e:                   # the floating-point grid has no int32 sums
        x = synth.normal((64, 64), 1.0, 1, device="cuda")
        q = srq.QSpec(8, format=srq.GRID_E4M3)
        srq.qlinear_fwd_ex(x, x, q, q, sums)
    assert e.value.status == binding.ERR_UNSUPPORTED
