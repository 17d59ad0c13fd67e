"""libmate: multi-view (row / column / prefix) sparse attention for flattened tables on B200.

Thin Python binding over the C ABI declared in include/mate.h.  Every step of the path runs in the
CUDA library; this package only marshals arguments (torch is used for device memory and streams).
"""
from .api import (  # noqa: F401
    MateError, Plan, mate_plan, mate_plan_bucketed, mate_plan_varlen, mate_plan_packed, mate_plan_sat,
    mate_plan_bucketed_global, mate_attn_fwd, mate_attn_bwd, mate_attn_bwd_noalloc,
    mate_attn_workspace_bytes, mate_cell_mean,
    library_path, IMPL_AUTO, IMPL_SIMT, IMPL_TCGEN05, FLAG_VIEW_ORDER, FLAG_BULK_TILES, FLAG_GATHER_TILES, VIEW_ROW, VIEW_COL,
)
