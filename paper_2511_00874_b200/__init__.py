"""B200-native stochastically-rounded quantized linear layer.

The product is the C-ABI library ``libsrq.so`` (hand-written CUDA for sm_100a, declared in
``include/srq.h``); this package holds its sources (``csrc/``), the build step (``build.py``),
a thin ctypes binding with the same entry-point names (``binding.py``) and the seeded synthetic
input recipes (``synth.py``).  Importing the package loads nothing; the first call loads the
library and raises if it has not been built.
"""
from .binding import (Output, qlinear_bwd_ex, qlinear_fwd_ex, srq_gemm_i8_ex,  # noqa: F401
                      BF16, F32, GRID_E4M3, GRID_INT, GRID_NONE, PER_ROW, PER_TENSOR, RTN, SR, SR8, DebugOut, QSpec, SrqError,  # noqa: F401
                      launch_count, new_workspace, qlinear_bwd, qlinear_bwd_input, qlinear_bwd_weight,
                      qlinear_fwd, sr_quantize, sr_quantize_static, srq_absmax, srq_absmax_cols, srq_dequant_i32, srq_gemm_e4m3, srq_gemm_i8, srq_gemm_workspace_bytes,
                      srq_poll_status, srq_quantize_workspace_bytes, srq_selftest_bounded_wait, srq_selftest_mma_rate, srq_set_product_timer, new_product_timer, srq_workspace_bytes,
                      status_string)
