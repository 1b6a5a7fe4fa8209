"""Small conveniences on top of the binding: size a configuration from a tree's arrays and
load whole-tree K/V into the pools.  No arithmetic of the method lives here."""
from __future__ import annotations

from typing import Optional

import numpy as np

from .binding import EtsContext, make_config


def bounds_for_tree(parent, cap_tokens, leaf_node, page_size: int = 16):
    """(n_nodes, n_leaves, max path capacity in tokens, sum of path lengths in nodes, pages)."""
    parent = np.asarray(parent, dtype=np.int64)
    cap = np.asarray(cap_tokens, dtype=np.int64)
    leaf_node = np.asarray(leaf_node, dtype=np.int64)
    n = parent.shape[0]
    cum_tok = np.zeros(n, np.int64)
    cum_nodes = np.zeros(n, np.int64)
    for i in range(n):
        p = parent[i]
        cum_tok[i] = cap[i] + (cum_tok[p] if p >= 0 else 0)
        cum_nodes[i] = 1 + (cum_nodes[p] if p >= 0 else 0)
    max_path_tokens = int(cum_tok[leaf_node].max()) if leaf_node.size else 1
    path_entries = int(cum_nodes[leaf_node].sum()) if leaf_node.size else 1
    pages = int(((cap + page_size - 1) // page_size).sum())
    return n, int(leaf_node.shape[0]), max(max_path_tokens, 1), max(path_entries, 1), max(pages, 1)


def context_for_tree(num_q_heads: int, num_kv_heads: int, head_dim: int, parent, cap_tokens, leaf_node, *,
                     num_layers: int = 1, device: int = 0, extra_pages: int = 0,
                     max_append_tokens: int = 0, sm_scale: float = 0.0,
                     chunk_pages: Optional[int] = None) -> EtsContext:
    n, l, mpt, mpe, pages = bounds_for_tree(parent, cap_tokens, leaf_node)
    cfg = make_config(num_q_heads, num_kv_heads, head_dim, num_layers=num_layers, max_nodes=max(n, 1),
                      max_leaves=max(l, 1), max_path_tokens=mpt, max_path_entries=mpe,
                      pages_per_layer=pages + extra_pages, max_append_tokens=max_append_tokens,
                      device=device, sm_scale=sm_scale)
    ctx = EtsContext(cfg)
    if chunk_pages is not None:
        from .binding import ETS_OPT_CHUNK_PAGES
        ctx.set_option(ETS_OPT_CHUNK_PAGES, chunk_pages)
    return ctx
