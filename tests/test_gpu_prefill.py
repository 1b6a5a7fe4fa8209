"""GPU parity of step-prefill attention (ets_tree_attn_prefill) against the fp64 oracle: every token of a
newly generated step is a leaf on the step's node, sees its ancestors whole and its own step causally."""
import numpy as np
import pytest
import torch

import paper_2502_13575_b200 as ets
from paper_2502_13575_b200.runner import context_for_tree
from oracle.tree_attention import tree_prefill_attention
from workloads import Geometry, make_workload, random_small_tree, node_kv_bits, query_bits
from _harness import node_values, fill_layer, bits_to_dev, dev_to_bits, check_close

pytestmark = pytest.mark.gpu


def _steps_as_leaves(tree, step_nodes, new_tokens):
    """Leaves and limits for the last new_tokens[i] tokens of every node in step_nodes."""
    leaves, limits = [], []
    for n, t_new in zip(step_nodes, new_tokens):
        length = int(tree.tokens[n])
        for j in range(t_new):
            leaves.append(int(n))
            limits.append(length - t_new + j + 1)
    return np.array(leaves, np.int32), np.array(limits, np.int32)


def _run(tree, geom, seed, leaves, limits, *, wide, sample, qscale=1.0, check_lse=True, path_items=False):
    ctx = context_for_tree(geom.num_q_heads, geom.num_kv_heads, geom.head_dim, tree.parent, tree.tokens, leaves)
    ctx.set_option(ets.ETS_OPT_WIDE, wide)
    ctx.set_option(ets.ETS_OPT_PATH_ITEMS, int(path_items))
    ctx.tree_build(tree.parent, tree.tokens, leaves)
    ks, vs = node_values(tree, geom, seed, 0)
    fill_layer(ctx, 0, ks, vs)
    L = leaves.shape[0]
    qb = query_bits(seed, 0, L, geom.num_q_heads, geom.head_dim, qscale)
    q = bits_to_dev(qb)
    out = torch.empty_like(q)
    lse = torch.empty((L, geom.num_q_heads), dtype=torch.float32, device="cuda")
    lim = torch.from_numpy(limits).cuda()
    ctx.tree_attn_prefill(0, q, lim, out, lse)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref, ref_lse = tree_prefill_attention(tree.parent, tree.tokens, leaves, limits, ks, vs, qb,
                                          geom.num_q_heads, geom.num_kv_heads, leaves=sample)
    check_close(dev_to_bits(out)[sample], ref[sample], "prefill")
    if check_lse:
        got = lse.cpu().numpy().astype(np.float64)[sample]
        assert np.all(np.abs(got - ref_lse[sample]) <= 1e-3 + 1e-3 * np.abs(ref_lse[sample]))
    return ctx, q, lim, out


@pytest.mark.parametrize("wide,path_items", [(17, False), (65, False), (17, True)])
def test_last_step_of_a_width16_tree(wide, path_items):
    """All tokens of the last search step of cfg2 (16 nodes of 64..128 tokens) as queries: 1.5k leaves whose
    groups are dense (256..512 rows on their own node, thousands on the shared ancestors)."""
    wl = make_workload("cfg2")
    tree, g = wl.tree, wl.geometry
    step_nodes = sorted(set(int(n) for n in tree.leaf_node))
    leaves, limits = _steps_as_leaves(tree, step_nodes, [int(tree.tokens[n]) for n in step_nodes])
    rng = np.random.default_rng(1)
    first_of_steps = np.flatnonzero(limits == 1)[:3].tolist()
    sample = sorted(set([0, leaves.shape[0] - 1] + first_of_steps + [int(x) for x in rng.integers(0, leaves.shape[0], size=10)]))
    ctx, q, lim, out = _run(tree, g, wl.value_seed, leaves, limits, wide=wide, sample=sample, path_items=path_items)
    if path_items:
        # one partial per (query, kv head), and the decode entry point refuses a tree built this way
        st = ctx.get_stats()
        assert st["n_partial_slots"] == leaves.shape[0] * g.num_kv_heads
        with pytest.raises(ets.EtsError) as e:
            ctx.tree_attn_decode(0, q, out, None)
        assert e.value.code == ets.ETS_ERR_STATE


def test_partial_steps_short_steps_and_peaked_scores():
    """Steps of which only the last few tokens are new (the node already held a prefix), steps of one to three
    tokens (at most 12 rows: the scalar kernel's items), limits that end inside a page, and peaked softmax."""
    wl = make_workload("cfg2")
    tree, g = wl.tree, wl.geometry
    nodes = sorted(set(int(n) for n in tree.leaf_node))
    new = [1, 2, 3, 17, 33, 5, 64, 16] + [int(tree.tokens[n]) // 2 for n in nodes[8:]]
    leaves, limits = _steps_as_leaves(tree, nodes, new)
    sample = list(range(0, leaves.shape[0], max(1, leaves.shape[0] // 24)))
    for qscale, path_items in ((1.0, False), (6.0, False), (1.0, True), (6.0, True)):
        _run(tree, g, wl.value_seed, leaves, limits, wide=17, sample=sample, qscale=qscale, path_items=path_items)


def test_full_limits_equal_decode_and_random_small_trees():
    """With every limit at its node's length the call is tree-decode attention (same bits as the decode entry
    point on the same build); random small trees, including internal-node steps and G = 1, 8."""
    rng = np.random.default_rng(5)
    for geom in (Geometry(8, 8, 64), Geometry(16, 2, 128), Geometry(4, 1, 64)):
        for _ in range(4):
            tree = random_small_tree(rng, max_nodes=9, max_tokens=70, allow_forest=True, allow_empty_nodes=False)
            nodes = sorted(set(int(n) for n in tree.leaf_node))
            new = [int(rng.integers(1, tree.tokens[n] + 1)) for n in nodes]
            leaves, limits = _steps_as_leaves(tree, nodes, new)
            sample = list(range(leaves.shape[0]))
            _run(tree, geom, 77, leaves, limits, wide=17, sample=sample, path_items=True)
            ctx, q, lim, out = _run(tree, geom, 77, leaves, limits, wide=17, sample=sample)
            full = torch.from_numpy(tree.tokens[leaves].astype(np.int32)).cuda()
            out_p, out_d = torch.empty_like(q), torch.empty_like(q)
            ctx.tree_attn_prefill(0, q, full, out_p, None)
            ctx.set_option(ets.ETS_OPT_KERNEL, 0)
            ctx.tree_attn_decode(0, q, out_d, None)
            torch.cuda.synchronize()
            ctx.poll_status()
            # different kernels serve the narrow items in the two calls: equal within twice the parity bar
            excess = ((out_p.float() - out_d.float()).abs() - (4e-3 + 2e-2 * out_d.float().abs())).max().item()
            assert excess <= 0, excess


@pytest.mark.parametrize("path_items", [False, True])
def test_limits_of_zero_and_beyond_the_node(path_items):
    """A limit of 0 hides the own node entirely (only ancestors are seen; at a root: nothing, which gives zeros
    and lse = -inf); a limit beyond the node's length is clipped to it."""
    geom = Geometry(8, 2, 128)
    parent = np.array([-1, 0, 0], np.int32)
    tokens = np.array([40, 33, 20], np.int32)
    from workloads import Tree
    tree = Tree(parent, tokens, np.array([1, 2], np.int32))
    #        leaf node:  root  root  1    1    1     2    2
    leaves = np.array([0, 0, 1, 1, 1, 2, 2] * 3, np.int32)          # 21 leaves: dense groups
    limits = np.array([0, 7, 0, 33, 99, 1, 20] * 3, np.int32)
    ctx = context_for_tree(geom.num_q_heads, geom.num_kv_heads, geom.head_dim, parent, tokens, leaves)
    ctx.set_option(ets.ETS_OPT_WIDE, 17)
    ctx.set_option(ets.ETS_OPT_PATH_ITEMS, int(path_items))
    ctx.tree_build(parent, tokens, leaves)
    ks, vs = node_values(tree, geom, 5, 0)
    fill_layer(ctx, 0, ks, vs)
    qb = query_bits(5, 0, leaves.shape[0], geom.num_q_heads, geom.head_dim)
    q = bits_to_dev(qb)
    out = torch.empty_like(q)
    lse = torch.empty((leaves.shape[0], geom.num_q_heads), dtype=torch.float32, device="cuda")
    ctx.tree_attn_prefill(0, q, torch.from_numpy(limits).cuda(), out, lse)
    torch.cuda.synchronize()
    ctx.poll_status()
    blind = np.flatnonzero((leaves == 0) & (limits == 0))
    assert np.all(dev_to_bits(out)[blind] == 0) and np.all(np.isneginf(lse.cpu().numpy()[blind]))
    seeing = [i for i in range(leaves.shape[0]) if i not in set(blind.tolist())]
    clipped = np.minimum(limits, tokens[leaves])
    ref, ref_lse = tree_prefill_attention(parent, tokens, leaves, clipped, ks, vs, qb, geom.num_q_heads, geom.num_kv_heads,
                                          leaves=seeing)
    check_close(dev_to_bits(out)[seeing], ref[seeing], "limits")
    got = lse.cpu().numpy().astype(np.float64)[seeing]
    assert np.all(np.abs(got - ref_lse[seeing]) <= 1e-3 + 1e-3 * np.abs(ref_lse[seeing]))
