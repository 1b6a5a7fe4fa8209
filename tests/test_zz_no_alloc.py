"""The allocation-free decode entry point (ets_tree_attn_decode_static).

Who needs it: code embedded in an application that owns the GPU memory budget, or a latency
critical loop where an allocation call is forbidden because it can stall the whole device.  Such a
caller cannot give the library a workspace for its intermediate partial results, so the library
keeps a fixed 8 MiB array of its own for them.

This file is collected last on purpose: if the entry point misbehaves, a run that stops at the
first failure has already exercised everything else.  It must also pass on its own in a fresh
process (the first call on a device performs the address lookup of the built-in array).
"""
import numpy as np
import pytest
import torch

import paper_2502_13575_b200 as ets
from paper_2502_13575_b200.runner import context_for_tree
from workloads import make_workload, query_bits
from _harness import node_values, fill_layer, bits_to_dev, dev_to_bits, check_close, ABS_TOL, REL_TOL
from oracle.tree_attention import tree_decode_attention, bf16_bits_to_f64

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice():
    wl = make_workload("cfg2")
    g, tree = wl.geometry, wl.tree
    ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, tree.tokens, tree.leaf_node)
    ctx.tree_build(tree.parent, tree.tokens, tree.leaf_node)
    ks, vs = node_values(tree, g, wl.value_seed, 0)
    fill_layer(ctx, 0, ks, vs)
    L = tree.n_leaves
    for call in range(2):   # two calls in a row: the second one finds the first one's leftovers
        qb = query_bits(wl.value_seed, 40 + call, L, g.num_q_heads, g.head_dim)
        q = bits_to_dev(qb)
        out_ws = torch.empty_like(q)
        lse_ws = torch.empty((L, g.num_q_heads), dtype=torch.float32, device="cuda")
        ctx.tree_attn_decode(0, q, out_ws, lse_ws)
        out_st = torch.full_like(q, float("nan"))
        lse_st = torch.full_like(lse_ws, float("nan"))
        ctx.tree_attn_decode_static(0, q, out_st, lse_st)
        torch.cuda.synchronize()
        ctx.poll_status()
        a = bf16_bits_to_f64(dev_to_bits(out_ws))
        b = bf16_bits_to_f64(dev_to_bits(out_st))
        assert np.all(np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(a)), f"call {call}"
        assert torch.allclose(lse_st, lse_ws, rtol=1e-3, atol=1e-3)
        # and both agree with the oracle
        ref, _ = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, ks, vs, qb,
                                       g.num_q_heads, g.num_kv_heads)
        check_close(dev_to_bits(out_st), ref, f"static call {call}")


def test_static_scratch_rejects_trees_beyond_its_size():
    wl = make_workload("cfg5b")      # ~3.6k partial slots x 8 rows x 520 B: beyond 8 MiB
    g, tree = wl.geometry, wl.tree
    ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, tree.tokens, tree.leaf_node)
    ctx.tree_build(tree.parent, tree.tokens, tree.leaf_node)
    st = ctx.get_stats()
    assert st["n_partial_slots"] * g.gqa * (g.head_dim + 2) * 4 > 8 << 20
    q = torch.zeros((tree.n_leaves, g.num_q_heads, g.head_dim), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    with pytest.raises(ets.EtsError) as e:
        ctx.tree_attn_decode_static(0, q, out, None)
    assert e.value.code == ets.ETS_ERR_POOL_EXHAUSTED
    assert "built-in scratch" in str(e.value)
