"""B200-native VECTOR hot path: thin Python binding over the C-ABI CUDA library.

The package holds the CUDA sources (``csrc/``), the in-tree build of
``libvector.so`` and a ctypes binding whose functions carry the same names as
the C entry points.  PyTorch is used only for device memory and streams.
"""
from .binding import (  # noqa: F401
    VectorError, Shape, Budget, Cache,
    VECTOR_F32, VECTOR_BF16,
    load_library, library_path,
    vector_status_string, vector_plan_budget, vector_calibrate, vector_workspace_bytes,
    vector_score, vector_score_keydiff, vector_pool_select, vector_residual, vector_truncate, vector_route,
    vector_compact, vector_diagnostics, DIAG_FIELDS, vector_decode_attn, alloc_cache, alloc_workspace,
    vector_layer_workspace_bytes, vector_layer_scores, vector_residual_layer, vector_route_layer, vector_compact_layer,
    vector_decode_attn_layer,
    vector_r2_global, vector_r2_global_workspace_bytes, R2_FIELDS, vector_sync_check,
    vector_device_fault, vector_kernel_launches, vector_decode_attn_static, vector_decode_scratch_bytes, VECTOR_STATIC_SCRATCH_BYTES,
)
