"""B200-native LOCKS decode hot path: thin ctypes binding over liblocks.so (C ABI in include/locks.h).

Argument marshalling only -- every step of the path runs in the CUDA kernels of the library.
PyTorch supplies device memory and streams.  Importing this package never builds or falls back:
if liblocks.so is missing, `lib()` raises.
"""
from .binding import (  # noqa: F401
    BF16, F32, FMT_F32, FMT_I4, FMT_I8, FMT_BF16, PARTITION_AUTO, PARTITION_BALANCED, PARTITION_STRIDED,
    COMBINE_SHARE_AVG, COMBINE_GROUP_MAX, COMBINE_GROUP_MASS, COMBINE_PER_HEAD, SCORER_SUMMARY, SCORER_CENTROID, SCORER_MOMENT,
    SCORER_ENVELOPE, Config, KV, LocksError, Context, lib, library_path,
    locks_summary_bytes, locks_workspace_bytes, locks_strerror, locks_sparse_attend_noalloc,
)
