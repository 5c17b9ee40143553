"""B200-native layer-wise structured-OBS solver of ZipLM (arXiv 2302.04089, Sec. 3.1).

The compute lives in ``libziplm.so`` (hand-written CUDA for sm_100a behind a C ABI, declared in
``include/ziplm.h``); :mod:`paper_2302_04089_b200.binding` is a thin ctypes layer with the same
names.  torch is used for device memory and streams only.
"""
from .binding import (  # noqa: F401
    ZiplmError, Status, lib_path, load_library, hessian_accumulate, hessian_accumulate_tokens,
    hessian_tokens_workspace_bytes, damped_inverse, damped_inverse_noalloc, prune_layers,
    status_string, hessian_workspace_bytes, inverse_workspace_bytes, prune_workspace_bytes,
    kept_structures, gather_columns, gather_rows, select_levels, select_workspace_bytes,
    search_levels, search_workspace_bytes, Option, set_option, get_option, launch_count, profile_begin, profile_end, profile_phase_count, profile_phase_name,
)
