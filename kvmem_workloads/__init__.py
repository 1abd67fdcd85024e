"""Seeded synthetic KV workspaces shaped like the paper's 128K-1M-token agent histories.

This package only draws inputs (keys, values, queries, planted-block ids, page tables).
It contains none of the method's arithmetic and imports neither the CPU oracle nor the
CUDA library; both are fed from here so that they see identical bytes.
"""
from .synth import (  # noqa: F401
    CONFIGS,
    WorkloadSpec,
    kv_blocks,
    make_queries,
    page_table,
    planted_blocks,
    planted_directions,
    select_params,
)
