"""B200-native suffix-automaton drafting and greedy verification (C-ABI library + thin binding).

Importing this package does not load the CUDA library; the first call does, and it raises
if the library has not been built (``python -m paper_2512_18337_b200.build``) or cannot be
loaded.  There is no CPU fallback.
"""
from .binding import (  # noqa: F401
    SamError,
    SamIndex,
    exported_symbols,
    library_path,
    sam_build,
    sam_build_growing,
    sam_extend,
    sam_pending,
    sam_renormalize,
    sam_sync,
    sam_update_stats,
    sam_draft,
    sam_export,
    sam_free,
    sam_last_cuda_error,
    sam_launch_count,
    sam_profile_count,
    sam_profile_enable,
    sam_profile_read,
    sam_set_argmax_variant,
    sam_sizes,
    sam_step,
    sam_step_host,
    sam_step_host_staging_bytes,
    sam_strerror,
    sam_upload,
    sam_verify,
    sam_verify_static,
    sam_workspace_bytes,
    sam_workspace_init,
    sam_workspace_status,
)
