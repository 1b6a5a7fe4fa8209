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


def test_static_decode_after_pipelined_host_step_without_a_join():
    """Like every device entry point, the allocation-free decode first joins host-buffer calls that are still in
    flight on the library's own streams.  Here a pipelined ets_decode_step_host (which appends one token per leaf)
    is followed directly by the static decode on the caller's stream, with no ets_host_join in between: the
    static decode has to see the appended tokens, and the two must not share the attention kernel's item queue
    at the same time.  Checked against the oracle on the grown tree, three rounds in a row."""
    wl = make_workload("cfg2")
    g, tree = wl.geometry, wl.tree
    L = tree.n_leaves
    rounds = 3
    cap = tree.tokens.copy()
    cap[tree.leaf_node] += rounds
    ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, cap, tree.leaf_node)
    ctx.tree_build(tree.parent, cap, tree.leaf_node)
    ks, vs = node_values(tree, g, wl.value_seed, 0)
    fill_layer(ctx, 0, ks, vs)
    ctx.set_option(ets.ETS_OPT_HOST_PIPELINE, 1)
    rng = np.random.default_rng(17)
    lengths = tree.tokens.copy()
    keep_alive = []
    for r in range(rounds):
        kb = rng.integers(0, 1 << 16, size=(L, g.num_kv_heads, g.head_dim), dtype=np.uint16) & np.uint16(0xBFFF)
        vb = rng.integers(0, 1 << 16, size=(L, g.num_kv_heads, g.head_dim), dtype=np.uint16) & np.uint16(0xBFFF)
        qb_h = query_bits(wl.value_seed, 60 + r, L, g.num_q_heads, g.head_dim)
        k_h = torch.from_numpy(kb.view(np.int16)).pin_memory()
        v_h = torch.from_numpy(vb.view(np.int16)).pin_memory()
        q_h = torch.from_numpy(qb_h.view(np.int16)).pin_memory()
        out_h = torch.empty_like(q_h).pin_memory()
        keep_alive.append((k_h, v_h, q_h, out_h))
        ctx.decode_step_host(0, k_h, v_h, q_h, out_h, None)          # returns without joining
        qb = query_bits(wl.value_seed, 80 + r, L, g.num_q_heads, g.head_dim)
        q = bits_to_dev(qb)
        out = torch.full_like(q, float("nan"))
        ctx.tree_attn_decode_static(0, q, out, None)                 # no ets_host_join before it
        torch.cuda.synchronize()
        ctx.poll_status()
        for i, n in enumerate(tree.leaf_node):
            ks[n] = np.concatenate([ks[n], kb[i][None]])
            vs[n] = np.concatenate([vs[n], vb[i][None]])
        lengths[tree.leaf_node] += 1
        ref, _ = tree_decode_attention(tree.parent, lengths, tree.leaf_node, ks, vs, qb, g.num_q_heads, g.num_kv_heads)
        check_close(dev_to_bits(out), ref, f"static decode after host step, round {r}")
        ref_h, _ = tree_decode_attention(tree.parent, lengths, tree.leaf_node, ks, vs, qb_h, g.num_q_heads, g.num_kv_heads)
        check_close(out_h.numpy().view(np.uint16), ref_h, f"host step, round {r}")
