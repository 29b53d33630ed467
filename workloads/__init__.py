"""Seeded synthetic DETOX workloads (inputs only; none of the aggregation arithmetic lives here).

The CUDA library and the CPU oracle are both fed from this module and from nothing else in common.
"""
from .gen import (  # noqa: F401
    CONFIGS,
    RESNET18_D,
    RESNET50_D,
    VGG_D,
    Workload,
    WorkloadSpec,
    expected_byzantine_votes,
    MeanEstimation,
    make_groups,
    make_mean_estimation,
    make_sets,
    make_workload,
    padded_ld,
    place_byzantine,
    sweep_legs,
    sweep_specs,
)
