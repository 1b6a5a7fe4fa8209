"""The seeded generators: determinism, the shapes the configs call for, and the KV-sharing
ratio of the diverse / ETS-like pair (the paper's 1.8x figure, Table 2)."""
import numpy as np
import pytest

from workloads import (CONFIG_NAMES, make_workload, tree_stats, node_kv_bits, query_bits,
                       f32_to_bf16_bits, bf16_bits_to_f32, layer_transform_bits)
from workloads import trees as wt


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e38], dtype=np.float32)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    got = bf16_bits_to_f32(f32_to_bf16_bits(x))
    assert got.tolist()[:4] == [1.0, 1.0, 1.015625, -1.0]
    import torch
    y = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    tb = torch.from_numpy(y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(f32_to_bf16_bits(y), tb)


SINGLE_TREES = [n for n in CONFIG_NAMES if not n.startswith("forest")]


@pytest.mark.parametrize("name,width,steps", [("forest_w16x8", 16, 4), ("forest_w64x8", 64, 8)])
def test_forest_shapes(name, width, steps):
    """Eight concurrent problems in one parent array: eight roots, eight times the width, no edge between problems."""
    t = make_workload(name).tree
    assert int((t.parent == -1).sum()) == 8 and t.n_leaves == 8 * width
    assert all(-1 <= int(p) < i for i, p in enumerate(t.parent))
    root_of = np.arange(t.n_nodes)
    for i, p in enumerate(t.parent):
        if p >= 0:
            root_of[i] = root_of[p]
    roots = root_of[t.leaf_node]
    assert [int((roots == r).sum()) for r in np.unique(roots)] == [width] * 8
    st = tree_stats(t)
    assert st["max_depth"] == steps + 1 and st["path_nodes"] == 8 * width * (steps + 1)
    # the problems differ from one another
    sizes = [int(t.tokens[root_of == r].sum()) for r in np.unique(root_of)]
    assert len(set(sizes)) == 8


@pytest.mark.parametrize("name", SINGLE_TREES)
def test_tree_shapes(name):
    wl = make_workload(name)
    t = wl.tree
    st = tree_stats(t)
    width = {"cfg1": 8, "cfg2": 16, "cfg3_diverse": 64, "cfg3_ets": 64, "cfg4": 256,
             "cfg5a": 128, "cfg5b": 128, "cfg5c": 128}[name]
    steps = {"cfg1": 3, "cfg2": 4, "cfg3_diverse": 8, "cfg3_ets": 8, "cfg4": 12,
             "cfg5a": 6, "cfg5b": 6, "cfg5c": 6}[name]
    assert t.n_leaves == width
    assert st["max_depth"] == steps + 1 and st["path_nodes"] == width * (steps + 1)
    assert all(-1 <= int(p) < i for i, p in enumerate(t.parent))
    assert int((t.parent == -1).sum()) == 1
    # every node has a live leaf below it
    alive = np.zeros(t.n_nodes, bool)
    for leaf in t.leaf_node:
        v = int(leaf)
        while v >= 0:
            alive[v] = True
            v = int(t.parent[v])
    assert alive.all()


def test_fixed_sizes():
    assert tree_stats(make_workload("cfg1").tree)["unique_tokens"] == 256
    assert tree_stats(make_workload("cfg5a").tree)["unique_tokens"] == 18048
    assert tree_stats(make_workload("cfg5b").tree)["unique_tokens"] == 99328
    assert make_workload("cfg1").tree.n_nodes == 15


def test_ets_pair_ratio():
    d = tree_stats(make_workload("cfg3_diverse").tree)["unique_tokens"]
    e = tree_stats(make_workload("cfg3_ets").tree)["unique_tokens"]
    assert 1.7 <= d / e <= 1.9
    assert make_workload("cfg3_ets").notes["kv_ratio_vs_diverse"] == pytest.approx(d / e)


def test_determinism_and_prefix_property():
    wt._CACHE.clear()
    a = make_workload("cfg2").tree
    wt._CACHE.clear()
    b = make_workload("cfg2").tree
    assert np.array_equal(a.parent, b.parent) and np.array_equal(a.tokens, b.tokens)
    k1, v1 = node_kv_bits(7, 3, 10, 2, 8)
    k2, v2 = node_kv_bits(7, 3, 25, 2, 8)
    assert np.array_equal(k1, k2[:10]) and np.array_equal(v1, v2[:10])
    assert not np.array_equal(k1, v1)
    k3, _ = node_kv_bits(7, 4, 10, 2, 8)
    assert not np.array_equal(k1, k3)
    # layers: rotation + sign flip, exact
    kl, _ = node_kv_bits(7, 3, 10, 2, 8, layer=3)
    assert np.array_equal(kl, layer_transform_bits(k1, 3))
    assert np.array_equal(bf16_bits_to_f32(kl), -np.roll(bf16_bits_to_f32(k1), 3, axis=-1))
    q0 = query_bits(7, 0, 4, 4, 8)
    q1 = query_bits(7, 1, 4, 4, 8)
    assert q0.shape == (4, 4, 8) and not np.array_equal(q0, q1)


def test_values_look_standard_normal():
    k, v = node_kv_bits(11, 0, 4096, 2, 64)
    x = bf16_bits_to_f32(k).astype(np.float64)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01


def _row_set(bits):
    return {r.tobytes() for r in bits.reshape(-1, bits.shape[-1])}


def test_queries_share_no_row_with_any_node():
    """The query stream has a key of its own: on cfg2 no query row of any of the first layers equals a K or V
    row of any node in that layer (they once shared node 2's key, which peaked every softmax below it)."""
    wl = make_workload("cfg2")
    g, tree = wl.geometry, wl.tree
    for layer in (0, 1, 2):
        kv_rows = set()
        for n in range(tree.n_nodes):
            k, v = node_kv_bits(wl.value_seed, n, int(tree.tokens[n]), g.num_kv_heads, g.head_dim, layer)
            kv_rows |= _row_set(k) | _row_set(v)
        q = query_bits(wl.value_seed, layer, tree.n_leaves, g.num_q_heads, g.head_dim)
        assert not (_row_set(q) & kv_rows)
    # the deliberately aligned variant is what the name says: its rows are node 2's K rows
    qa = query_bits(wl.value_seed, 0, tree.n_leaves, g.num_q_heads, g.head_dim, aligned_with_node2=True)
    k2, _ = node_kv_bits(wl.value_seed, 2, int(tree.tokens[2]), g.num_kv_heads, g.head_dim, 0)
    n = min(qa.size, k2.size)
    assert np.array_equal(qa.reshape(-1)[:n], k2.reshape(-1)[:n])


def test_queries_look_standard_normal_and_unpeaked():
    """With independent N(0,1) queries the scores q.k/sqrt(d) are N(0,1): no leaf of cfg2 sees a score near
    |q|^2/sqrt(d) = 11."""
    from workloads import bf16_bits_to_f32 as f32
    wl = make_workload("cfg2")
    g, tree = wl.geometry, wl.tree
    q = f32(query_bits(wl.value_seed, 0, tree.n_leaves, g.num_q_heads, g.head_dim)).astype(np.float64)
    assert abs(q.mean()) < 0.02 and abs(q.std() - 1.0) < 0.02
    k2, _ = node_kv_bits(wl.value_seed, 2, int(tree.tokens[2]), g.num_kv_heads, g.head_dim, 0)
    s = np.einsum("lad,thd->lath", q, f32(k2).astype(np.float64)) / np.sqrt(g.head_dim)
    assert np.abs(s).max() < 6.0
