"""GPU parity of the three layer passes (Alg. 1 and Alg. 2) against the CPU oracle:
codes, step sizes and int32 sums bit for bit, fp32 outputs equal (0 ulp; bound 1 ulp)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import synth

pytestmark = pytest.mark.gpu

PASSES = {
    "fwd": (srq.qlinear_fwd, oracle.qlinear_fwd),
    "bwd_input": (srq.qlinear_bwd_input, oracle.qlinear_bwd_input),
    "bwd_weight": (srq.qlinear_bwd_weight, oracle.qlinear_bwd_weight),
}


def _ulp_diff(a, b):
    ia = a.view(np.int32).astype(np.int64)
    ib = b.view(np.int32).astype(np.int64)
    ia = np.where(ia < 0, -(ia & 0x7FFFFFFF), ia)
    ib = np.where(ib < 0, -(ib & 0x7FFFFFFF), ib)
    return np.abs(ia - ib).max() if a.size else 0


def run_pass(name, X0, X1, T, N, K, q0, q1, ws=None, full=True):
    """Runs one pass on the GPU and in the oracle; returns (gpu out tensor, oracle result)."""
    fn, ofn = PASSES[name]
    dev = X0.device
    shapes = {"fwd": ((T, K), (N, K), (T, N)), "bwd_input": ((T, N), (K, N), (T, K)),
              "bwd_weight": ((N, T), (K, T), (N, K))}[name]
    n_a = shapes[0][0] if q0.scale == srq.PER_ROW else 1
    n_b = shapes[1][0] if q1.scale == srq.PER_ROW else 1
    out = torch.full(shapes[2], float("nan"), device=dev)
    dbg = srq.DebugOut(torch.empty(shapes[0], dtype=torch.int8, device=dev), torch.empty(n_a, device=dev),
                       torch.empty(shapes[1], dtype=torch.int8, device=dev), torch.empty(n_b, device=dev),
                       torch.empty(shapes[2], dtype=torch.int32, device=dev))
    if ws is None:
        ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K), dev)
    fn(X0, X1, q0, q1, out, dbg, ws)
    st = srq.srq_poll_status(ws)
    assert st == 0, srq.status_string(st)
    oq = lambda q: oracle.QSpec(q.bits, q.scale, q.round, q.seed, q.tensor_id, q.index_offset)
    ref = ofn(X0.float().cpu().numpy(), X1.float().cpu().numpy(), oq(q0), oq(q1))
    if full:
        assert np.array_equal(dbg.codes_a.cpu().numpy(), ref.codes_a), name + ": codes of first operand"
        assert np.array_equal(dbg.codes_b.cpu().numpy(), ref.codes_b), name + ": codes of second operand"
        assert np.array_equal(dbg.scale_a.cpu().numpy(), ref.scale_a), name + ": step sizes of first operand"
        assert np.array_equal(dbg.scale_b.cpu().numpy(), ref.scale_b), name + ": step sizes of second operand"
        assert np.array_equal(dbg.acc.cpu().numpy(), ref.acc), name + ": int32 sums"
        o = out.cpu().numpy()
        assert _ulp_diff(o, ref.out) <= 1, name + ": fp32 output beyond 1 ulp"
        assert np.array_equal(o, ref.out), name + ": fp32 output"
        # the same call without the debug copies (the product then stores whole blocks): same output
        out2 = torch.full(shapes[2], float("nan"), device=dev)
        fn(X0, X1, q0, q1, out2, None, ws)
        assert srq.srq_poll_status(ws) == 0
        assert np.array_equal(out2.cpu().numpy(), ref.out), name + ": fp32 output without debug copies"
    return out, ref


def layer_specs(scale, rnd, seed, bits_fwd=8, bits_bwd=8):
    # five quantization points per layer: A and W forward; A, W and dY backward
    return {"a_fwd": srq.QSpec(bits_fwd, scale, rnd, seed, 0), "w_fwd": srq.QSpec(bits_fwd, scale, rnd, seed, 1),
            "a_bwd": srq.QSpec(bits_bwd, scale, rnd, seed, 2), "w_bwd": srq.QSpec(bits_bwd, scale, rnd, seed, 3),
            "dy_bwd": srq.QSpec(bits_bwd, scale, rnd, seed, 4)}


def all_passes(A, W, dY, q, ws=None):
    T, K = A.shape
    N = W.shape[0]
    run_pass("fwd", A, W, T, N, K, q["a_fwd"], q["w_fwd"], ws)
    run_pass("bwd_input", dY, W, T, N, K, q["dy_bwd"], q["w_bwd"], ws)
    run_pass("bwd_weight", dY, A, T, N, K, q["dy_bwd"], q["a_bwd"], ws)


def test_single_layer_8bit_per_tensor_seed0():
    """A 64x256, W 256x256, dY 64x256 fp32, 8-bit per-tensor SR, seed 0."""
    A, W, dY = synth.layer_inputs(64, 256, 256, seed=0, device="cuda", std_dy=1.0)
    all_passes(A, W, dY, layer_specs(srq.PER_TENSOR, srq.SR, 0))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
@pytest.mark.parametrize("rnd", [srq.SR, srq.RTN])
def test_ragged_multi_tile_layer(dtype, scale, rnd):
    T, N, K = 264, 392, 328            # all three differ, none a tile multiple
    A, W, dY = synth.layer_inputs(T, N, K, seed=1, dtype=dtype, device="cuda", std_dy=1e-3)
    all_passes(A, W, dY, layer_specs(scale, rnd, seed=3, bits_fwd=8, bits_bwd=4))


def test_odd_extents_take_the_elementwise_path():
    T, N, K = 37, 21, 50
    A, W, dY = synth.layer_inputs(T, N, K, seed=2, device="cuda")
    all_passes(A, W, dY, layer_specs(srq.PER_ROW, srq.SR, seed=9, bits_bwd=6))


def test_gpt2_shaped_layer_small_batch():
    """GPT-2-small projection 768 -> 2304 at 1024 tokens; 64 sampled rows per output."""
    T, K, N = 1024, 768, 2304
    A, W, dY = synth.layer_inputs(T, N, K, seed=3, device="cuda", std_dy=1e-3)
    all_passes(A, W, dY, layer_specs(srq.PER_TENSOR, srq.SR, seed=0))


def test_workspace_reuse_and_shared_quantized_weight():
    """One workspace for all passes; the same (seed, tensor_id) for W forward and backward
    gives one quantized W, its backward layout being the transpose of the forward one."""
    T, N, K = 256, 384, 512
    A, W, dY = synth.layer_inputs(T, N, K, seed=4, device="cuda")
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    q = layer_specs(srq.PER_TENSOR, srq.SR, seed=1)
    q["w_bwd"] = q["w_fwd"]
    dev = A.device
    cw = torch.empty((N, K), dtype=torch.int8, device=dev)
    cwt = torch.empty((K, N), dtype=torch.int8, device=dev)
    Y = torch.empty((T, N), device=dev)
    dA = torch.empty((T, K), device=dev)
    srq.qlinear_fwd(A, W, q["a_fwd"], q["w_fwd"], Y, srq.DebugOut(codes_b=cw), ws)
    srq.qlinear_bwd_input(dY, W, q["dy_bwd"], q["w_bwd"], dA, srq.DebugOut(codes_b=cwt), ws)
    assert srq.srq_poll_status(ws) == 0
    assert torch.equal(cw.t(), cwt)
    all_passes(A, W, dY, q, ws)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scale", [srq.PER_TENSOR, srq.PER_ROW])
@pytest.mark.parametrize("shape", [(264, 392, 328), (37, 21, 50), (512, 256, 384)])
def test_whole_backward_pass_in_one_call(dtype, scale, shape):
    """qlinear_bwd (Alg. 2 as one call, dY read once) against the oracle's two backward products:
    codes of all four operands, step sizes, int32 sums and outputs bit for bit."""
    T, N, K = shape
    A, W, dY = synth.layer_inputs(T, N, K, seed=5, dtype=dtype, device="cuda", std_dy=1e-3)
    q = layer_specs(scale, srq.SR, seed=2, bits_fwd=8, bits_bwd=6)
    dev = A.device
    per_row = scale == srq.PER_ROW
    n = lambda rows: rows if per_row else 1
    dA = torch.full((T, K), float("nan"), device=dev)
    dW = torch.full((N, K), float("nan"), device=dev)
    di = srq.DebugOut(torch.empty((T, N), dtype=torch.int8, device=dev), torch.empty(n(T), device=dev),
                      torch.empty((K, N), dtype=torch.int8, device=dev), torch.empty(n(K), device=dev),
                      torch.empty((T, K), dtype=torch.int32, device=dev))
    dw = srq.DebugOut(torch.empty((N, T), dtype=torch.int8, device=dev), torch.empty(n(N), device=dev),
                      torch.empty((K, T), dtype=torch.int8, device=dev), torch.empty(n(K), device=dev),
                      torch.empty((N, K), dtype=torch.int32, device=dev))
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K), dev)
    srq.qlinear_bwd(dY, A, W, q["dy_bwd"], q["a_bwd"], q["w_bwd"], dA, dW, di, dw, ws)
    assert srq.srq_poll_status(ws) == 0
    oq = lambda s: oracle.QSpec(s.bits, s.scale, s.round, s.seed, s.tensor_id, s.index_offset)
    f = lambda t: t.float().cpu().numpy()
    ri = oracle.qlinear_bwd_input(f(dY), f(W), oq(q["dy_bwd"]), oq(q["w_bwd"]))
    rw = oracle.qlinear_bwd_weight(f(dY), f(A), oq(q["dy_bwd"]), oq(q["a_bwd"]))
    for name, dbg, out, ref in (("dA", di, dA, ri), ("dW", dw, dW, rw)):
        assert np.array_equal(dbg.codes_a.cpu().numpy(), ref.codes_a), name + ": codes of first operand"
        assert np.array_equal(dbg.codes_b.cpu().numpy(), ref.codes_b), name + ": codes of second operand"
        assert np.array_equal(dbg.scale_a.cpu().numpy(), ref.scale_a), name + ": step sizes of first operand"
        assert np.array_equal(dbg.scale_b.cpu().numpy(), ref.scale_b), name + ": step sizes of second operand"
        assert np.array_equal(dbg.acc.cpu().numpy(), ref.acc), name + ": int32 sums"
        assert np.array_equal(out.cpu().numpy(), ref.out), name + ": fp32 output"
    # without debug copies (block-store epilogue), same outputs
    dA2, dW2 = torch.empty_like(dA), torch.empty_like(dW)
    srq.qlinear_bwd(dY, A, W, q["dy_bwd"], q["a_bwd"], q["w_bwd"], dA2, dW2, None, None, ws)
    assert srq.srq_poll_status(ws) == 0
    assert torch.equal(dA2, dA) and torch.equal(dW2, dW)


def test_overflowing_contraction_is_refused():
    A = torch.zeros((133145, 16), device="cuda")
    dY = torch.zeros((133145, 16), device="cuda")
    dW = torch.empty((16, 16), device="cuda")
    with pytest.raises(srq.SrqError) as e:
        srq.qlinear_bwd_weight(dY, A, srq.QSpec(8), srq.QSpec(8), dW)
    assert e.value.status == 4
    srq.qlinear_bwd_weight(dY, A, srq.QSpec(4), srq.QSpec(8), dW)       # 7 * 127 * T fits
    assert torch.count_nonzero(dW).item() == 0


def test_layer_with_eight_random_bits_per_element():
    T, N, K = 264, 400, 336
    A, W, dY = synth.layer_inputs(T, N, K, seed=6, device="cuda", std_dy=1e-3)
    all_passes(A, W, dY, layer_specs(srq.PER_TENSOR, srq.SR8, seed=4, bits_fwd=8, bits_bwd=4))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_operands_of_one_call_with_different_quantization_points(dtype):
    """Small layers quantize all operands of a call in one pair of launches; every operand keeps its own
    point there: per-row steps beside per-tensor steps, round-to-nearest beside 24-bit and 8-bit
    stochastic rounding, different widths, one operand with a maximum the caller already knows."""
    T, N, K = 136, 264, 328
    A, W, dY = synth.layer_inputs(T, N, K, seed=12, dtype=dtype, device="cuda", std_dy=1e-3)
    q = {"a_fwd": srq.QSpec(8, srq.PER_ROW, srq.SR, 5, 0), "w_fwd": srq.QSpec(5, srq.PER_TENSOR, srq.RTN, 5, 1),
         "a_bwd": srq.QSpec(6, srq.PER_TENSOR, srq.SR8, 5, 2), "w_bwd": srq.QSpec(8, srq.PER_ROW, srq.RTN, 5, 3),
         "dy_bwd": srq.QSpec(4, srq.PER_ROW, srq.SR, 5, 4)}
    all_passes(A, W, dY, q)
    # the whole backward pass in one call (three operands in the batch), A's maximum handed in
    m = torch.zeros(1, device="cuda")
    srq.srq_absmax(A, m)
    qa = srq.QSpec(6, srq.PER_TENSOR, srq.SR8, 5, 2, absmax=m)
    dA, dW = torch.empty((T, K), device="cuda"), torch.empty((N, K), device="cuda")
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))
    srq.qlinear_bwd(dY, A, W, q["dy_bwd"], qa, q["w_bwd"], dA, dW, None, None, ws)
    assert srq.srq_poll_status(ws) == 0
    oq = lambda s: oracle.QSpec(s.bits, s.scale, s.round, s.seed, s.tensor_id, s.index_offset)
    f = lambda t: t.float().cpu().numpy()
    assert np.array_equal(dA.cpu().numpy(), oracle.qlinear_bwd_input(f(dY), f(W), oq(q["dy_bwd"]), oq(q["w_bwd"])).out)
    assert np.array_equal(dW.cpu().numpy(), oracle.qlinear_bwd_weight(f(dY), f(A), oq(q["dy_bwd"]), oq(q["a_bwd"])).out)
    # a non-finite input of any operand of the batch reaches the status word
    W2 = W.clone()
    W2[3, 5] = float("nan")
    srq.qlinear_bwd(dY, A, W2, q["dy_bwd"], qa, q["w_bwd"], dA, dW, None, None, ws)
    assert srq.srq_poll_status(ws) == srq.binding.ERR_NONFINITE


@pytest.mark.parametrize("case", range(16))
def test_random_layers(case):
    """Seeded random layers: extents (aligned and odd, rows long enough for the one-pass per-row
    quantizer included), input type, step-size mode, rounding mode, forward and backward widths."""
    rng = np.random.default_rng(300 + case)
    T = int(rng.choice([rng.integers(1, 300), 8 * rng.integers(4, 60)]))
    N = int(rng.choice([rng.integers(1, 300), 8 * rng.integers(4, 60)]))
    K = int(rng.choice([rng.integers(1, 300), 8 * rng.integers(4, 60), 1024]))
    dtype = [torch.float32, torch.bfloat16][int(rng.integers(2))]
    scale = [srq.PER_TENSOR, srq.PER_ROW][int(rng.integers(2))]
    rnd = [srq.SR, srq.RTN, srq.SR8][int(rng.integers(3))]
    A, W, dY = synth.layer_inputs(T, N, K, seed=case, dtype=dtype, device="cuda", std_dy=1e-3)
    q = layer_specs(scale, rnd, seed=case, bits_fwd=int(rng.integers(3, 9)), bits_bwd=int(rng.integers(2, 9)))
    all_passes(A, W, dY, q)


@pytest.mark.parametrize("scale,dtype", [(srq.PER_TENSOR, torch.float32), (srq.PER_ROW, torch.bfloat16)])
def test_a_layer_step_recorded_in_a_cuda_graph_replays_the_same_results(scale, dtype):
    """The calls only enqueue work on the caller's stream, so forward + backward can be recorded once in
    a CUDA graph (after one call outside the capture, which does the one-time device set-up) and
    replayed; the replay gives the oracle's results, again after the inputs have changed."""
    T, N, K = 264, 392, 1024
    q = layer_specs(scale, srq.SR, seed=3)
    A, W, dY = synth.layer_inputs(T, N, K, seed=1, dtype=dtype, device="cuda", std_dy=1e-3)
    Y, dA, dW = torch.empty((T, N), device="cuda"), torch.empty((T, K), device="cuda"), torch.empty((N, K), device="cuda")
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K))

    def step():
        srq.qlinear_fwd(A, W, q["a_fwd"], q["w_fwd"], Y, None, ws)
        srq.qlinear_bwd(dY, A, W, q["dy_bwd"], q["a_bwd"], q["w_bwd"], dA, dW, None, None, ws)

    step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    oq = lambda s: oracle.QSpec(s.bits, s.scale, s.round, s.seed, s.tensor_id, s.index_offset)
    f = lambda t: t.float().cpu().numpy()
    for rep in range(2):
        if rep == 1:                             # new inputs in the same buffers: the graph reads them at replay
            A2, W2, dY2 = synth.layer_inputs(T, N, K, seed=2, dtype=dtype, device="cuda", std_dy=1e-3)
            A.copy_(A2); W.copy_(W2); dY.copy_(dY2)
        for t in (Y, dA, dW):
            t.fill_(float("nan"))
        g.replay()
        assert srq.srq_poll_status(ws) == 0
        assert np.array_equal(Y.cpu().numpy(), oracle.qlinear_fwd(f(A), f(W), oq(q["a_fwd"]), oq(q["w_fwd"])).out)
        assert np.array_equal(dA.cpu().numpy(), oracle.qlinear_bwd_input(f(dY), f(W), oq(q["dy_bwd"]), oq(q["w_bwd"])).out)
        assert np.array_equal(dW.cpu().numpy(), oracle.qlinear_bwd_weight(f(dY), f(A), oq(q["dy_bwd"]), oq(q["a_bwd"])).out)
