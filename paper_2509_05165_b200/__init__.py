"""KVCompose compression pass for NVIDIA B200: thin Python binding over the C-ABI library.

Every step runs in the CUDA kernels of ``libkvc.so``; this package only marshals
arguments (torch tensors are used for device memory and streams).
"""
from .binding import (  # noqa: F401
    AGG_MAX,
    AGG_MEAN,
    BF16,
    F32,
    KvcDesc,
    KvcError,
    desc_from_config,
    kvc_allocate,
    kvc_allocate_static,
    kvc_budget_from_ratio,
    kvc_compose,
    kvc_compress,
    kvc_compress_unstructured,
    kvc_desc_init,
    kvc_gather,
    kvc_gather_unstructured,
    kvc_order_kept,
    kvc_last_error,
    kvc_launch_count,
    kvc_debug_score_hooks,
    kvc_score,
    kvc_score_status_offset,
    kvc_score_uses_tensor_cores,
    kvc_score_weighted,
    kvc_select_unstructured,
    kvc_version,
    kvc_workspace_size,
    library_path,
    CompressOutputs,
    compress,
)
