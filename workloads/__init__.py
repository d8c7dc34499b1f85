"""Seeded synthetic inputs shaped like the paper's workloads.

This package only manufactures inputs (gradient rows, clip radii, run settings).
It contains none of the aggregation or verification arithmetic and is the one
module that both the oracle-side tests and the GPU-side tests and benchmark use.
"""
from .synth import CONFIGS, Workload, make_workload, make_partition, layout_ceil_pad  # noqa: F401
