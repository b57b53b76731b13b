"""sr_quantize_static, the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (a fully assigned memory pool, a
plug-in that only ever receives its input and output tensors, a latency-critical loop), so this
variant keeps its scratch in an array built into the library.  The test calls it through the C
ABI twice in a row, without synchronising in between, and checks each result bit for bit against
sr_quantize (the tolerance of the quantizer parity tests: codes and step sizes exact).  The
second call uses a smaller input with smaller magnitudes, so anything the first call left in the
shared array (absmax words are combined with a maximum) would change its result.
"""
import ctypes

import pytest
import torch

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
    # 256 + 2 * (pad(rows) + pad(cols)) * 4 bytes > 1 MiB: refused on the host, nothing enqueued
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
