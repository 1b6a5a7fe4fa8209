"""Pins for the reference flattener: a hand-worked tree, and invariants that follow from
the tree/KV-sharing semantics (a node is on a leaf's path iff the leaf descends from it)."""
import numpy as np
import pytest

from oracle.flatten import ReferenceFlattener, BadTree, PoolExhausted
from workloads import random_small_tree, make_workload, tree_stats
from _golden import read_golden


def test_hand_worked_tree():
    g = read_golden("flatten_small_tree.txt")
    f = ReferenceFlattener(g["page_size"][0], g["pages_per_layer"][0])
    t = f.build(g["parent"], g["cap_tokens"], g["leaf_node"])
    for key in ("node_page_off", "page_ids", "node_leaf_off", "node_leaves", "leaf_path_off",
                "leaf_path", "leaf_path_pos", "node_depth"):
        assert t[key].dtype == np.int32
        assert t[key].tolist() == g[key], key
    assert t["node_len"].tolist() == [0] * 6


def _descends(parent, node, anc):
    v = node
    while v >= 0:
        if v == anc:
            return True
        v = parent[v]
    return False


def _check_invariants(tree, tables, page_size, cap):
    n, L = tree.n_nodes, tree.n_leaves
    parent = tree.parent.tolist()
    # pages: each node owns ceil(cap/page) ids, no id twice
    po, ids = tables["node_page_off"], tables["page_ids"]
    assert po[0] == 0 and po[-1] == len(ids)
    for i in range(n):
        assert po[i + 1] - po[i] == -(-int(cap[i]) // page_size)
    assert len(set(ids.tolist())) == len(ids)
    # groups by brute force: leaf l is in group(n) iff leaf_node[l] descends from n
    lo, lv = tables["node_leaf_off"], tables["node_leaves"]
    for i in range(n):
        want = [l for l in range(L) if _descends(parent, int(tree.leaf_node[l]), i)]
        assert lv[lo[i]:lo[i + 1]].tolist() == want
    # duality: sum of group sizes == sum of path lengths
    pth_o, pth, pos = tables["leaf_path_off"], tables["leaf_path"], tables["leaf_path_pos"]
    assert lo[-1] == pth_o[-1]
    for l in range(L):
        path = pth[pth_o[l]:pth_o[l + 1]].tolist()
        assert path[-1] == int(tree.leaf_node[l])
        assert parent[path[0]] == -1
        for a, b in zip(path[:-1], path[1:]):
            assert parent[b] == a
        for v, p in zip(path, pos[pth_o[l]:pth_o[l + 1]].tolist()):
            assert lv[lo[v] + p] == l
    depth = tables["node_depth"]
    for i in range(n):
        assert depth[i] == (0 if parent[i] < 0 else depth[parent[i]] + 1)


def test_invariants_on_random_trees():
    rng = np.random.default_rng(21)
    for _ in range(200):
        tree = random_small_tree(rng)
        f = ReferenceFlattener(4, 256)
        t = f.build(tree.parent, tree.tokens, tree.leaf_node)
        _check_invariants(tree, t, 4, tree.tokens)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3_ets", "cfg5a"])
def test_invariants_on_configs(name):
    wl = make_workload(name)
    st = tree_stats(wl.tree)
    f = ReferenceFlattener(16, 1 << 16)
    t = f.build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node)
    _check_invariants(wl.tree, t, 16, wl.tree.tokens)
    # single root: the root's group is every leaf
    assert t["node_leaf_off"][1] - t["node_leaf_off"][0] == wl.tree.n_leaves
    assert t["leaf_path_off"][-1] == st["path_nodes"]
    # fresh pool, ascending allocation: page ids are 0..P-1 in order
    assert t["page_ids"].tolist() == list(range(len(t["page_ids"])))


def test_sharing_inequality():
    # sum over leaves of path tokens >= unique tokens, equal for a chain-free split at an empty root
    for name in ("cfg2", "cfg3_diverse", "cfg5a", "cfg5b"):
        st = tree_stats(make_workload(name).tree)
        assert st["path_tokens"] >= st["unique_tokens"]
    f = ReferenceFlattener(4, 64)
    t = f.build([-1, 0, 0, 0], [0, 5, 6, 7], [1, 2, 3])
    assert t["node_page_off"].tolist() == [0, 0, 2, 4, 6]


def test_keep_pages_and_heap_order():
    f = ReferenceFlattener(4, 10)
    t0 = f.build([-1, 0, 0], [8, 4, 8], [1, 2])          # pages: n0 {0,1} n1 {2} n2 {3,4}
    assert t0["page_ids"].tolist() == [0, 1, 2, 3, 4]
    f.append(0, 8)
    f.append(2, 5)
    # new tree: old node 2 becomes node 1 and keeps its pages; old node 1 is dropped (page 2 freed);
    # node 0 kept but now needs 3 pages; a new node 2 needs 2 pages.
    t1 = f.build([-1, 0, 1], [12, 8, 5], [2], keep_pages_of=[0, 2, -1])
    # free heap after release: {2,5,6,7,8,9}; node0 keeps {0,1} + pops 2; node1 keeps {3,4}; node2 pops 5,6
    assert t1["node_page_off"].tolist() == [0, 3, 5, 7]
    assert t1["page_ids"].tolist() == [0, 1, 2, 3, 4, 5, 6]
    assert t1["node_len"].tolist() == [8, 5, 0]
    # shrinking a kept node releases its tail pages and clips its length
    t2 = f.build([-1], [3], [0], keep_pages_of=[0])
    assert t2["page_ids"].tolist() == [0]
    assert t2["node_len"].tolist() == [3]
    t3 = f.build([-1, 0], [4, 4], [1])
    assert t3["page_ids"].tolist() == [0, 1]


def test_errors_leave_state_untouched():
    f = ReferenceFlattener(4, 4)
    f.build([-1, 0], [4, 4], [1])
    with pytest.raises(BadTree):
        f.build([0, -1], [4, 4], [1])           # parent after child
    with pytest.raises(BadTree):
        f.build([-1, 0], [4, -1], [1])
    with pytest.raises(BadTree):
        f.build([-1, 0], [4, 4], [2])
    with pytest.raises(BadTree):
        f.build([-1, 0], [4, 4], [1], keep_pages_of=[0, 0])
    with pytest.raises(PoolExhausted):
        f.build([-1, 0], [12, 12], [1])
    # still the first tree
    assert f.node_pages == [[0], [1]]
    with pytest.raises(PoolExhausted):
        f.append(1, 5)
    assert f.append(1, 4) == 0


def test_empty_tree():
    f = ReferenceFlattener(16, 8)
    t = f.build([], [], [])
    assert t["node_page_off"].tolist() == [0] and t["leaf_path_off"].tolist() == [0]
