"""B200-native swizzled tiled GEMM: Python face of libswizzleperf.so.

``tile_map`` returns the remap of tile ids, ``gemm`` runs the bf16 GEMM under it; both are
thin wrappers over the C ABI declared in ``include/swizzleperf.h``.  All computation runs
in hand-written sm_100a kernels; nothing here falls back to another implementation.
"""

from .binding import (  # noqa: F401
    COL_MAJOR, CUSTOM, DIE_SPLIT, GROUP_M, GROUP_N, HILBERT, HILBERT_RECT, MORTON, ROW_MAJOR, XCD, SCHEME_NAMES,
    ERR_ALIGNMENT, ERR_CUDA, ERR_DEVICE, ERR_INVALID_ARG, ERR_NOT_BIJECTIVE, ERR_TIMEOUT, ERR_UNSUPPORTED, OK,
    SpError, SpParams, gemm, gemm_host, gemm_noalloc, gemm_trace, gemm_units, get_status, last_error, lib, make_params, probe_dispatch, probe_l2_capacity, probe_topology, selftest_timeout,
    shutdown, recommend, streamk_plan, FLAG_DIE_PINNED, FLAG_SERPENTINE, FLAG_STREAM_K, FLAG_OVERLAP, FLAG_CLC, FLAG_K_ALTERNATE, FLAG_STEAL, FLAG_HINT_C_EVICT_FIRST, FLAG_HINT_A_EVICT_FIRST, FLAG_HINT_B_EVICT_FIRST, FLAG_HINT_A_EVICT_LAST, FLAG_HINT_B_EVICT_LAST, WORK_FULL, WORK_CONTRIB, WORK_OWNER, tile_count, tile_map, tile_map_device, transpose, stencil2d, STENCIL_TILE, softmax, SOFTMAX_TILE, SOFTMAX_SINGLE_PASS, SOFTMAX_TWO_PHASE, SOFTMAX_TWO_PHASE_REVERSED,
)
