"""fp64 CPU oracle for the BlossomRec sparse-attention path.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()``
and by ``bench.py``'s CPU-baseline / reference arm.  The product package never
imports it, and this package never imports the product.
"""
from .blossom_oracle import (  # noqa: F401
    build,
    forward,
    backward,
    forward_backward,
    select_blocks, select_blocks_cmp, select_blocks_gqa, select_blocks_per_query, rope, forward_gqa, backward_gqa,
    threads,
)
