"""B200-native AMPNet training engine: thin Python binding of the C ABI in include/ampnet.h.

Every step of the hot path runs in the CUDA library (libampnet.so); this package only marshals
arguments.  PyTorch supplies device memory (through the allocator callbacks) and the CUDA stream.
There is no CPU fallback: without the built library or without a CUDA device the calls raise.
"""
from .binding import Engine, EpochStats, AmpnetError, load_library, RunCfg, ir_tables, measure_fma_peak  # noqa: F401
