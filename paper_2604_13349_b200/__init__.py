"""B200-native relay-boundary prompt-KV compression (headwise eviction + Orthogonal BackFill).

The product is the C-ABI CUDA library declared in ``include/obf.h``; this package
holds its sources (``csrc/``), the in-tree build step, a ctypes binding with the
same entry-point names, and the seeded synthetic input generator.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    OBF_BF16, OBF_F32, OBF_OK, ObfCache, ObfDiag, ObfError, ObfParams, compress_caches, evict_only, evict_only_static, obf_static_scratch_status,
    load, make_cache, make_params, obf_compress, obf_compress_host, obf_compress_profiled, obf_host_arena_bytes,
    obf_last_device_status, obf_last_launch_count, obf_status_string, obf_workspace_bytes, parse_diag)
