"""Forward pass with unquantized bfloat16 activations and a quantized weight (the Sec. 3.3 variant,
D_A^fwd = 0) against the oracle's binary64 product, within 1e-5 * |row| * |col| (the product runs
in bfloat16 on the tensor cores with binary32 accumulation)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,N,K", [(64, 256, 256), (264, 392, 328), (1, 8, 8), (1024, 2304, 768), (300, 40, 4096)])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
def test_forward_with_unquantized_activations(T, N, K, scale):
    A, W, _ = synth.layer_inputs(T, N, K, seed=7, dtype=torch.bfloat16, device="cuda")
    qa = srq.QSpec(format=srq.GRID_NONE)
    qw = srq.QSpec(8, scale, srq.SR, 5, 1)
    Y = torch.full((T, N), float("nan"), device="cuda")
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    srq.qlinear_fwd(A, W, qa, qw, Y, None, ws)
    assert srq.srq_poll_status(ws) == 0
    hA, hW = A.float().cpu().numpy(), W.float().cpu().numpy()
    ref = oracle.qlinear_fwd_fp_act(hA, hW, oracle.QSpec(8, scale, oracle.SR, 5, 1))
    # the same quantized weight as the fully quantized forward pass with this quantization point
    cw = torch.empty((N, K), dtype=torch.int8, device="cuda")
    sw = torch.empty(N if scale == srq.PER_ROW else 1, device="cuda")
    srq.sr_quantize(W, qw, cw, sw)
    assert np.array_equal(cw.cpu().numpy(), ref.codes_b) and np.array_equal(sw.cpu().numpy(), ref.scale_b)
    sc = np.broadcast_to(ref.scale_b.astype(np.float64), (N,))
    bound = 1e-5 * np.linalg.norm(hA.astype(np.float64), axis=1)[:, None] * (np.linalg.norm(ref.codes_b.astype(np.float64), axis=1) * sc)[None, :]
    err = np.abs(Y.cpu().numpy().astype(np.float64) - ref.out)
    assert np.all(err <= bound + np.abs(ref.out) * 2e-7 + 1e-30)


def test_requirements_are_checked_on_the_host():
    A32, W32, _ = synth.layer_inputs(16, 16, 16, seed=1, device="cuda")
    Y = torch.empty((16, 16), device="cuda")
    with pytest.raises(srq.SrqError) as e:                      # fp32 activations are not fed to the tensor cores
        srq.qlinear_fwd(A32, W32, srq.QSpec(format=srq.GRID_NONE), srq.QSpec(8), Y)
    assert e.value.status == 2
    A, W, _ = synth.layer_inputs(16, 16, 12, seed=1, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(srq.SrqError) as e:                      # rows of A must start on 16-byte boundaries
        srq.qlinear_fwd(A, W, srq.QSpec(format=srq.GRID_NONE), srq.QSpec(8), Y)
    assert e.value.status == 1
    with pytest.raises(srq.SrqError):                           # only the first operand of the forward pass
        dY = synth.normal((16, 16), 1.0, 2, torch.bfloat16, "cuda")
        srq.qlinear_bwd_input(dY, W, srq.QSpec(format=srq.GRID_NONE), srq.QSpec(8), torch.empty((16, 12), device="cuda"))
