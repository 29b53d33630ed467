"""DETOX parameter-server gradient aggregation on NVIDIA B200 (sm_100a).

The product is the C-ABI library built from csrc/ (include/detox.h); this package is its Python binding.
"""
from .binding import (  # noqa: F401
    AGG_BULYAN,
    AGG_COORD_MEDIAN,
    AGG_GEOMETRIC_MEDIAN,
    AGG_MEAN,
    AGG_MULTIKRUM,
    AGG_NONE,
    AGG_TRIMMED_MEAN,
    EXPORTS,
    LIB_PATH,
    DetoxError,
    Pipeline,
    agg_bulyan,
    agg_bulyan_workspace_bytes,
    agg_coord_median,
    agg_coord_median_workspace_bytes,
    agg_geometric_median,
    agg_multikrum,
    agg_trimmed_mean,
    agg_multikrum_workspace_bytes,
    detox_aggregate,
    detox_aggregate_workspace_bytes,
    detox_hier_mean,
    detox_vote,
    detox_vote_hier_mean,
    detox_vote_noalloc,
    detox_vote_workspace_bytes,
    load,
    status_string,
)
