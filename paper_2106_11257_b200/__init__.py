"""Batched CenteredClip + verification for one NVIDIA B200 (sm_100a).

The arithmetic lives in ``libbtard.so`` (hand-written CUDA behind a C ABI, see ``include/btard.h``);
this package is the ctypes binding.  There is no CPU fallback: importing works anywhere, but every
call needs the compiled library and a CUDA device.
"""
from .binding import (  # noqa: F401
    INIT_CALLER_V0, INIT_ZERO, INIT_MEAN, INIT_COORD_MEDIAN, ALGO_DIRECT, ALGO_GRAM, ALGO_DIRECT_COOPERATIVE,
    STOP_FIXED_ITERS, STOP_EPS, RULE_CENTERED_CLIP, RULE_GEOMETRIC_MEDIAN, RULE_MEAN, RULE_COORD_MEDIAN, SPLIT_PAPER, SPLIT_CEIL_PAD, STATUS_NOT_CONVERGED,
    STATUS_NONFINITE_ROW, BtardError, lib, library_path, partition_layout, centered_clip,
    centered_clip_workspace, verify_projections, verify_projections_workspace, random_vector,
    aggregate_host, aggregate_host_scratch, kernel_launch_count, last_cuda_error, EXPORTS,
    profile_enable, profile_collect, KERNEL_KINDS, verify_projections_static, verification_checks, preclip, centered_clip_verify, split_gradients, merge_partitions, hash_partitions,
)
