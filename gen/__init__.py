"""Seeded synthetic inputs for the Hotline hot path.

This package only *draws inputs* (table geometry, sparse index batches, dense
features, initial table values, upstream gradients).  It holds none of the
method's arithmetic: no counting, no hot-set selection, no fragmenting, no
pooling, no update.  Both the CPU oracle's tests and the CUDA path's tests feed
on these arrays; neither of those two imports the other.
"""
from .synthetic import (  # noqa: F401
    CONFIGS,
    Batch,
    Geometry,
    WorkloadSpec,
    feistel_permute,
    grad_values,
    make_batch,
    make_geometry,
    mix32,
    restrict_to_rows,
    table_values,
    table_values_torch,
    zipf_ranks,
)
