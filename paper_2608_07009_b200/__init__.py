"""B200-native HiSparse selection resolution: CUDA library + thin binding.

`hisparse`  — binding of the C-ABI (include/hisparse.h); all compute runs in `_hisparse.so`.
`inputs`    — seeded synthetic histories and selection traces (no cache arithmetic).
`build`     — in-tree nvcc build of the library for sm_100a.
"""
from . import build, inputs  # noqa: F401
from .hisparse import (  # noqa: F401
    HiSparse, HostHistory, HiSparseError, ExternalState, resolve_noalloc, host_link_probe, scatter_read_probe, device_bytes, lib,
    FLAG_SKIP_IO, FLAG_DEBUG_VALIDATE, FLAG_INLINE_WRITE_THROUGH, FLAG_PHASE_TIMERS, FLAG_NO_PDL, FLAG_EAGER_ORDER, FLAG_WIDE_BLOCKS, FLAG_NARROW_BLOCKS,
    POLICY_LRU, POLICY_FIFO, POLICY_RANDOM,
    STATUS_OUT_OF_RANGE, STATUS_DUPLICATE, STATUS_CAPACITY, STATUS_INCONSISTENT, STATUS_TIMEOUT,
)
