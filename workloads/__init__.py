"""Seeded synthetic search trees and bf16 K/V/Q values.

This package only *draws inputs*: tree topologies, token counts and normally
distributed values rounded to bf16.  It contains none of the attention
arithmetic and none of the table-flattening rules, so both the CUDA library's
tests and the CPU oracle's tests can be fed from it without sharing any of the
method's code.
"""
from .trees import (  # noqa: F401
    Geometry,
    Tree,
    Workload,
    CONFIG_NAMES,
    make_workload,
    random_small_tree,
    tree_stats,
)
from .search import SEARCH_NAMES, run_search, make_search_workload  # noqa: F401
from .values import (  # noqa: F401
    f32_to_bf16_bits,
    bf16_bits_to_f32,
    layer_transform_bits,
    node_kv_bits,
    query_bits,
    TOPOLOGY_SEED_BASE,
    VALUE_SEED_BASE,
)
