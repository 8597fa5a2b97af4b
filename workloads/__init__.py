"""Seeded synthetic parameter sets shaped like the paper's workloads.

This package only draws random inputs (live parameters ``x``, running
checkpoint ``z``, block geometry, lost-set masks).  It holds none of the
method's arithmetic: no distances, no selection, no packing, no norms.  Both
the CPU oracle's tests and the CUDA path's tests/benchmark take their inputs
from here so that the two sides always see byte-identical data.
"""

from .configs import (  # noqa: F401
    CONFIGS,
    Geometry,
    Workload,
    make_workload,
    block_offsets,
    shard_block_ranges,
    bylayer_offsets,
    make_cnn_bylayer,
)
