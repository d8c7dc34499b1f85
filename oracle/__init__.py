"""Float64 CPU oracle for batched CenteredClip and its verification pass.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg, never by the GPU library or its Python binding.
The arithmetic lives in ``btard_oracle.c`` (plain C, double precision); this
module compiles it with gcc and marshals numpy arrays to it.  Nothing here is
shared with the CUDA path.
"""
from .oracle import (  # noqa: F401
    INIT_CALLER, INIT_ZERO, INIT_MEAN, INIT_COORD_MEDIAN, STOP_FIXED, STOP_EPS,
    SPLIT_PAPER, SPLIT_CEIL_PAD, RULE_CENTERED_CLIP, RULE_GEOMETRIC_MEDIAN, RULE_MEAN, RULE_COORD_MEDIAN, STATUS_NOT_CONVERGED, STATUS_NONFINITE_ROW,
    build, philox4x32_10, random_vector, partition_layout, centered_clip, verify,
    max_threads, checks, preclip, sha256, commitment,
)
