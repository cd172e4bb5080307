"""Python binding of the streaming decoder step's C-ABI library (libdc.so).

Argument marshalling only: every step of the decoder runs inside the CUDA
library.  torch is used for device memory and streams.  There is no fallback:
if the library is missing or no sm_100 device is present, calls raise.
"""
from .binding import (DCError, NOALLOC_SCRATCH_FLOATS, conv_stack_noalloc, Model, Stream, decode_batch, decode_batch_host, decode_wavefront_batch, library_path, load_library,  # noqa: F401
                      make_config, selftest_bounded_wait, STATUS, OPT_NO_GRAPH, OPT_NO_PDL, OPT_NO_ZEROCOPY, OPT_SERIAL_TAILS, OPT_ROUNDED_NORM, OPT_GUARD_ZONES, fail_allocation, measure_fp32_peak,
                      OPT_SKIP_CONV_GEMM, OPT_SKIP_ATTENTION, OPT_EMPTY_KERNELS, OPT_CTA_PAIRS)
