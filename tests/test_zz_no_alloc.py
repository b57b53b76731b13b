"""sr_quantize_static, the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (a fully assigned memory pool, a
plug-in that only ever receives its input and output tensors, a latency-critical loop), so this
variant keeps its scratch in an array built into the library.  The test calls it through the C
ABI twice in a row, without synchronising in between, and checks each result bit for bit against
sr_quantize and against the CPU oracle (the tolerance of the quantizer parity tests: codes and
step sizes exact).  The second call uses a smaller input with smaller magnitudes, so anything the
first call left in the shared array (absmax words are combined with a maximum) would change its
result.  Further cases walk the other routes through the entry point (one-pass per-row kernel,
given maxima, the floating-point grid, 8 random bits) and check that a call changes neither the
free device memory nor torch's allocation count.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2511_00874_b200 as srq
from paper_2511_00874_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _outputs(rows, cols, per_row):
    dev = "cuda"
    return (torch.full((rows, cols), 99, dtype=torch.int8, device=dev),
            torch.full((rows if per_row else 1,), -1.0, device=dev),
            torch.full((cols, rows), 99, dtype=torch.int8, device=dev),
            torch.full((cols if per_row else 1,), -1.0, device=dev))


@pytest.mark.parametrize("scale", [srq.PER_ROW, srq.PER_TENSOR])
def test_two_calls_in_a_row_match_the_workspace_entry_point(scale):
    per_row = scale == srq.PER_ROW
    big = synth.with_outliers((300, 388), seed=21, device="cuda") * 8.0
    small = synth.normal((132, 260), 0.01, seed=22, dtype=torch.bfloat16, device="cuda")
    q1 = srq.QSpec(8, scale, srq.SR, seed=5, tensor_id=1)
    q2 = srq.QSpec(4, scale, srq.SR, seed=6, tensor_id=2)

    got1, got2 = _outputs(300, 388, per_row), _outputs(132, 260, per_row)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    srq.sr_quantize_static(big, q1, *got1, device_status=status)
    srq.sr_quantize_static(small, q2, *got2)            # status kept inside the built-in array
    torch.cuda.synchronize()
    assert status.item() == 0

    for x, q, got in ((big, q1, got1), (small, q2, got2)):
        want = _outputs(x.shape[0], x.shape[1], per_row)
        ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(*x.shape))
        srq.sr_quantize(x, q, *want, ws)
        assert srq.srq_poll_status(ws) == 0
        for name, g, w in zip(("codes_rm", "scale_rm", "codes_tr", "scale_tr"), got, want):
            assert torch.equal(g, w), name
        # and directly against the oracle
        oq = oracle.QSpec(q.bits, oracle.PER_ROW if per_row else oracle.PER_TENSOR, oracle.SR, q.seed, q.tensor_id)
        ref = oracle.sr_quantize(x.float().cpu().numpy(), oq, True, True)
        for name, g, w in zip(("codes_rm", "scale_rm", "codes_tr", "scale_tr"), got, ref):
            assert np.array_equal(g.cpu().numpy(), w), name + " against the oracle"


def _static_and_workspace(x, q, want_rm=True, want_tr=True):
    per_row = q.scale == srq.PER_ROW
    rows, cols = x.shape
    got, want = _outputs(rows, cols, per_row), _outputs(rows, cols, per_row)
    sel = lambda o: (o[0] if want_rm else None, o[1] if want_rm else None, o[2] if want_tr else None, o[3] if want_tr else None)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    srq.sr_quantize_static(x, q, *sel(got), device_status=status)
    ws = srq.new_workspace(srq.srq_quantize_workspace_bytes(rows, cols))
    srq.sr_quantize(x, q, *sel(want), ws)
    assert srq.srq_poll_status(ws) == 0 and status.item() == 0
    for name, g, w in zip(("codes_rm", "scale_rm", "codes_tr", "scale_tr"), got, want):
        assert torch.equal(g, w), name
    return got


def test_other_routes_through_the_entry_point():
    # one-pass per-row kernel (row-major codes only, rows of 1024 bfloat16 elements): touches no scratch
    xb = synth.with_outliers((64, 1024), seed=31, dtype=torch.bfloat16, device="cuda")
    q = srq.QSpec(8, srq.PER_ROW, srq.SR, seed=1, tensor_id=3)
    got = _static_and_workspace(xb, q, want_tr=False)
    ref = oracle.sr_quantize(xb.float().cpu().numpy(), oracle.QSpec(8, oracle.PER_ROW, oracle.SR, 1, 3), True, False)
    assert np.array_equal(got[0].cpu().numpy(), ref[0]) and np.array_equal(got[1].cpu().numpy(), ref[1])
    # a maximum the caller already knows (per tensor), and known column maxima (per row, both layouts)
    x = synth.with_outliers((300, 388), seed=32, device="cuda")
    m = torch.zeros(1, device="cuda")
    srq.srq_absmax(x, m)
    _static_and_workspace(x, srq.QSpec(6, srq.PER_TENSOR, srq.SR, seed=2, tensor_id=4, absmax=m))
    mc = torch.zeros(388, device="cuda")
    srq.srq_absmax_cols(x, mc)
    got = _static_and_workspace(x, srq.QSpec(8, srq.PER_ROW, srq.SR, seed=2, tensor_id=5, absmax=mc))
    ref = oracle.sr_quantize(x.cpu().numpy(), oracle.QSpec(8, oracle.PER_ROW, oracle.SR, 2, 5), True, True)
    for g, w in zip(got, ref):
        assert np.array_equal(g.cpu().numpy(), w)
    # the floating-point grid and stochastic rounding with 8 random bits
    got = _static_and_workspace(x, srq.QSpec(8, srq.PER_TENSOR, srq.SR, seed=3, tensor_id=6, format=srq.GRID_E4M3))
    ref = oracle.sr_quantize_e4m3(x.cpu().numpy(), oracle.QSpec(8, oracle.PER_TENSOR, oracle.SR, 3, 6), True, True)
    assert np.array_equal(got[0].cpu().numpy().view(np.uint8), ref[0]) and np.array_equal(got[1].cpu().numpy(), ref[1])
    x16 = synth.with_outliers((160, 400), seed=33, device="cuda")
    got = _static_and_workspace(x16, srq.QSpec(8, srq.PER_TENSOR, srq.SR8, seed=4, tensor_id=7))
    ref = oracle.sr_quantize(x16.cpu().numpy(), oracle.QSpec(8, oracle.PER_TENSOR, oracle.SR8, 4, 7), True, True)
    assert np.array_equal(got[0].cpu().numpy(), ref[0]) and np.array_equal(got[2].cpu().numpy(), ref[2])


def test_a_call_allocates_nothing():
    x = synth.normal((512, 640), 1.0, seed=34, device="cuda")
    c, ct = torch.empty((512, 640), dtype=torch.int8, device="cuda"), torch.empty((640, 512), dtype=torch.int8, device="cuda")
    s, stt = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    srq.sr_quantize_static(x, srq.QSpec(), c, s, ct, stt)      # the first call on a device looks up the array's address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for i in range(3):
        srq.sr_quantize_static(x, srq.QSpec(seed=i), c, s, ct, stt)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


def test_nonfinite_input_reaches_the_callers_status_word_and_is_cleared_again():
    x = synth.normal((64, 64), 1.0, seed=23, device="cuda")
    x[1, 2] = float("inf")
    c, s = torch.empty((64, 64), dtype=torch.int8, device="cuda"), torch.empty(1, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    srq.sr_quantize_static(x, srq.QSpec(), c, s, device_status=status)
    torch.cuda.synchronize()
    assert status.item() == binding.ERR_NONFINITE
    x[1, 2] = 0.5
    srq.sr_quantize_static(x, srq.QSpec(), c, s, device_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0


def test_inputs_beyond_the_built_in_scratch_are_refused():
    # 512 + 2 * (pad64(rows) + pad64(cols)) * 4 bytes > 1 MiB: refused on the host, nothing enqueued
    x = torch.empty((1, 140000), device="cuda")
    c = torch.empty((1, 140000), dtype=torch.int8, device="cuda")
    with pytest.raises(srq.SrqError) as e:
        srq.sr_quantize_static(x, srq.QSpec(), c, torch.empty(1, device="cuda"))
    assert e.value.status == binding.ERR_WORKSPACE
    # the same extents the other way round, passed as bare numbers (no storage is touched)
    q = binding.QSpec().c()
    st = binding.lib().sr_quantize_static(x.data_ptr(), binding.F32, 140000, 1, 1, ctypes.byref(q),
                                          c.data_ptr(), 1, x.data_ptr(), None, 0, None, None, None)
    assert st == binding.ERR_WORKSPACE
