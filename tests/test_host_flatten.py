"""Host logic of the library, no GPU needed: the shared library loads and exports every symbol
the header declares; its tables match the reference flattener bit for bit; its private work
decomposition covers every (page, kv head, leaf) exactly once."""
import os
import re

import numpy as np
import pytest

import paper_2502_13575_b200 as ets
from oracle.flatten import ReferenceFlattener, BadTree, PoolExhausted
from workloads import random_small_tree, make_workload, tree_stats, CONFIG_NAMES
from paper_2502_13575_b200.runner import bounds_for_tree
from _golden import read_golden

TABLE_KEYS = ("node_page_off", "page_ids", "node_leaf_off", "node_leaves", "leaf_path_off",
              "leaf_path", "leaf_path_pos", "node_depth", "node_len")


def host_ctx(hq=4, hkv=1, d=64, page_size=16, pages=4096, max_nodes=4096, max_leaves=512,
             max_path_tokens=8192, max_path_entries=8192, layers=1):
    cfg = ets.make_config(hq, hkv, d, num_layers=layers, max_nodes=max_nodes, max_leaves=max_leaves,
                          max_path_tokens=max_path_tokens, max_path_entries=max_path_entries,
                          pages_per_layer=pages, page_size=page_size, device=-1)
    return ets.EtsContext(cfg)


def test_header_symbols_are_exported(repo_root):
    text = open(os.path.join(repo_root, "include", "ets.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(ets_[a-z_]+)\s*\(", text))
    assert {"ets_tree_build", "ets_kv_append", "ets_tree_attn_decode"} <= declared
    for name in declared:
        assert hasattr(ets.lib, name), f"{name} declared in ets.h but not exported"
    assert ets.ets_version().startswith("ets-b200")


def test_config_struct_layout_matches_header():
    # a mis-declared ctypes struct would scramble these values on the C side
    cfg = ets.make_config(32, 8, 128, max_nodes=10, max_leaves=4, max_path_tokens=64, max_path_entries=40,
                          pages_per_layer=7, device=-1)
    k, v, w = ets.ets_pool_bytes(cfg)
    # each of the two buffers holds K and V of every other page: ceil(7 / 2) page pairs x 8 heads x 2 tiles
    assert k == v == 4 * 8 * 2 * 16 * 128 * 2
    bad = ets.make_config(32, 8, 96, max_nodes=10, max_leaves=4, max_path_tokens=64, max_path_entries=40,
                          pages_per_layer=7, device=-1)
    with pytest.raises(ets.EtsError) as e:
        ets.ets_pool_bytes(bad)
    assert e.value.code == ets.ETS_ERR_UNSUPPORTED


def test_hand_worked_tree_matches():
    g = read_golden("flatten_small_tree.txt")
    ctx = host_ctx(page_size=g["page_size"][0], pages=g["pages_per_layer"][0])
    ctx.tree_build(g["parent"], g["cap_tokens"], g["leaf_node"])
    t = ctx.tree_export()
    for key in TABLE_KEYS[:-1]:
        assert t[key].tolist() == g[key], key


def _assert_same_tables(ctx, ref_tables):
    got = ctx.tree_export()
    for key in TABLE_KEYS:
        assert got[key].dtype == np.int32
        assert np.array_equal(got[key], ref_tables[key]), key


@pytest.mark.parametrize("name", CONFIG_NAMES)
def test_tables_bit_exact_on_configs(name):
    wl = make_workload(name)
    g = wl.geometry
    ctx = host_ctx(g.num_q_heads, g.num_kv_heads, g.head_dim, pages=1 << 15, max_path_entries=1 << 14)
    ref = ReferenceFlattener(16, 1 << 15)
    ctx.tree_build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node)
    _assert_same_tables(ctx, ref.build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node))
    st = ctx.get_stats()
    assert st["n_nodes"] == wl.tree.n_nodes and st["n_leaves"] == wl.tree.n_leaves
    assert st["unique_tokens"] == 0  # nothing appended yet


def test_tables_bit_exact_on_random_trees_and_rebuilds():
    rng = np.random.default_rng(31)
    for trial in range(300):
        page = int(rng.choice([1, 3, 4, 16]))
        pages = int(rng.integers(8, 200))
        ctx = host_ctx(page_size=page, pages=pages)
        ref = ReferenceFlattener(page, pages)
        prev_n = 0
        for step in range(4):
            tree = random_small_tree(rng)
            keep = None
            if prev_n and rng.random() < 0.8:
                keep = np.full(tree.n_nodes, -1, np.int32)
                olds = rng.permutation(prev_n)[: tree.n_nodes]
                for i, o in enumerate(olds):
                    if rng.random() < 0.6:
                        keep[i] = o
            try:
                want = ref.build(tree.parent, tree.tokens, tree.leaf_node, keep)
            except PoolExhausted:
                with pytest.raises(ets.EtsError) as e:
                    ctx.tree_build(tree.parent, tree.tokens, tree.leaf_node, keep)
                assert e.value.code == ets.ETS_ERR_POOL_EXHAUSTED
                continue
            ctx.tree_build(tree.parent, tree.tokens, tree.leaf_node, keep)
            _assert_same_tables(ctx, want)
            prev_n = tree.n_nodes


def test_errors_and_unchanged_state():
    ctx = host_ctx(pages=4)
    ctx.tree_build([-1, 0], [16, 16], [1])
    before = ctx.tree_export()
    cases = [
        (([0, -1], [4, 4], [1]), ets.ETS_ERR_BAD_TREE),
        (([-1, 0], [4, -1], [1]), ets.ETS_ERR_BAD_TREE),
        (([-1, 0], [4, 4], [2]), ets.ETS_ERR_BAD_TREE),
        (([-1, 0], [4, 4], [-1]), ets.ETS_ERR_BAD_TREE),
        (([-1, 0], [48, 48], [1]), ets.ETS_ERR_POOL_EXHAUSTED),
    ]
    for args, code in cases:
        with pytest.raises(ets.EtsError) as e:
            ctx.tree_build(*args)
        assert e.value.code == code
    with pytest.raises(ets.EtsError) as e:
        ctx.tree_build([-1, 0], [4, 4], [1], keep_pages_of=[0, 0])
    assert e.value.code == ets.ETS_ERR_BAD_TREE
    with pytest.raises(ets.EtsError) as e:
        ctx.tree_build([-1, 0], [4, 4], [1], keep_pages_of=[5, -1])
    assert e.value.code == ets.ETS_ERR_BAD_TREE
    after = ctx.tree_export()
    for k in TABLE_KEYS:
        assert np.array_equal(before[k], after[k])
    # device calls on a host-only context are refused, not attempted
    with pytest.raises(ets.EtsError) as e:
        ctx.tree_attn_decode(0, 0, 0)
    assert e.value.code == ets.ETS_ERR_STATE
    with pytest.raises(ets.EtsError) as e:
        ctx.set_option(99, 1)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG


def test_capacity_bounds():
    ctx = host_ctx(max_nodes=3, max_leaves=2, max_path_entries=4)
    for args in (([-1, 0, 0, 0], [1] * 4, [1]), ([-1, 0], [1, 1], [1, 1, 1]), ([-1, 0, 1], [1, 1, 1], [2, 2])):
        with pytest.raises(ets.EtsError) as e:
            ctx.tree_build(*args)
        assert e.value.code == ets.ETS_ERR_POOL_EXHAUSTED


def test_empty_tree():
    ctx = host_ctx()
    ctx.tree_build([], [], [])
    t = ctx.tree_export()
    assert t["node_page_off"].tolist() == [0] and t["leaf_path_off"].tolist() == [0]
    w = ctx.work_export()
    assert w["item"].shape[0] == 0


def _check_work(ctx, tree, cap, hkv, gqa, page=16):
    t = ctx.tree_export()
    w = ctx.work_export()
    unit, item = w["unit"], w["item"]
    leaves_per_tile = max(1, 16 // gqa)
    covered = {}   # (page, head, leaf) -> slot
    for it in item:
        ub, uc, head, lb, nl, slot0, seg, _ = (int(x) for x in it)
        assert 1 <= nl <= max(1, 128 // gqa) and uc >= 1
        leaves = t["node_leaves"][lb:lb + nl].tolist()
        for u in range(ub, ub + uc):
            pg, node, tok0, _z = (int(x) for x in unit[u])
            # the unit really is that page of that node
            j = tok0 // page
            assert t["page_ids"][t["node_page_off"][node] + j] == pg
            # every leaf of the tile descends from the node
            grp = t["node_leaves"][t["node_leaf_off"][node]:t["node_leaf_off"][node + 1]].tolist()
            for i, l in enumerate(leaves):
                assert l in grp
                key = (pg, head, l)
                assert key not in covered
                covered[key] = slot0 + i
    # every page of every node on every leaf's path is covered for every head, and the slot
    # that holds it is listed for that leaf
    for l in range(tree.n_leaves):
        for h in range(hkv):
            k = l * hkv + h
            slots = w["leaf_slots"][w["leaf_slot_off"][k]:w["leaf_slot_off"][k + 1]].tolist()
            assert len(set(slots)) == len(slots)
            used = set()
            for v in t["leaf_path"][t["leaf_path_off"][l]:t["leaf_path_off"][l + 1]]:
                for pg in t["page_ids"][t["node_page_off"][v]:t["node_page_off"][v + 1]]:
                    assert (int(pg), h, l) in covered
                    used.add(covered[(int(pg), h, l)])
            assert used == set(slots)
    n_cov = sum((t["node_page_off"][v + 1] - t["node_page_off"][v]) *
                (t["node_leaf_off"][v + 1] - t["node_leaf_off"][v]) for v in range(tree.n_nodes)) * hkv
    assert len(covered) == n_cov
    # slots of different (chunk, leaf) never collide
    assert w["n_partial_slots"] >= (max(covered.values()) + 1 if covered else 0)


@pytest.mark.parametrize("chunk_pages", [0, 1, 2, 5])
def test_work_decomposition_covers_everything_once(chunk_pages):
    rng = np.random.default_rng(41)
    for _ in range(60):
        hkv = int(rng.choice([1, 2]))
        gqa = int(rng.choice([1, 4, 8]))
        ctx = host_ctx(hq=hkv * gqa, hkv=hkv, max_path_tokens=1 << 14)
        ctx.set_option(ets.ETS_OPT_CHUNK_PAGES, chunk_pages)
        tree = random_small_tree(rng, max_nodes=14, max_tokens=90, max_leaves=9)
        ctx.tree_build(tree.parent, tree.tokens, tree.leaf_node)
        _check_work(ctx, tree, tree.tokens, hkv, gqa)


@pytest.mark.parametrize("name", ["cfg2", "cfg3_ets", "cfg5a", "cfg5c", "forest_w16x8"])
def test_work_decomposition_on_configs(name):
    wl = make_workload(name)
    g = wl.geometry
    ctx = host_ctx(g.num_q_heads, g.num_kv_heads, g.head_dim, pages=1 << 15, max_path_entries=1 << 14)
    ctx.tree_build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node)
    _check_work(ctx, wl.tree, wl.tree.tokens, g.num_kv_heads, g.gqa)
    st = ctx.get_stats()
    assert st["n_segments"] <= wl.tree.n_nodes
    if name == "cfg5a":
        # the five shared chain steps fuse with the root: 1 shared segment + 128 private ones
        assert st["n_segments"] == 129


@pytest.mark.parametrize("name", ["cfg2", "cfg3_ets", "cfg3_diverse", "cfg4", "cfg5b"])
def test_narrow_queue_is_ordered_longest_first(name):
    """Narrow items form a queue: warp w starts with item w and the rest are claimed in index order, so
    the items are sorted by length (longest first), none is longer than 32 page slots (one lane each),
    the late ones are short, and the static first assignment is one item per warp."""
    wl = make_workload(name)
    g = wl.geometry
    ctx = host_ctx(g.num_q_heads, g.num_kv_heads, g.head_dim, pages=1 << 15, max_path_entries=1 << 14)
    ctx.tree_build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node)
    w = ctx.work_export()
    off, item = w["worker_off"], w["item"]
    n_workers = len(off) - 1
    n_narrow = ctx.get_stats()["n_narrow_items"]
    assert off.tolist() == [min(k, n_narrow) for k in range(n_workers + 1)]
    narrow = item[:n_narrow]
    # items after the narrow queue are the wide ones (tiles of groups with more than 16 query rows)
    assert np.all(narrow[:, 4] * g.gqa <= 16)
    lens = narrow[:, 1]
    assert lens.max() <= 32 and lens.min() >= 1
    assert np.all(np.diff(lens) <= 0)
    if n_narrow > 2 * n_workers:
        # the pieces claimed last are at most half as long as the longest
        assert lens[-n_workers // 2:].max() * 2 <= max(lens.max(), 2) + 1
    # pieces of one (segment part) for all heads and leaf tiles are adjacent in the queue
    key = [(int(r[6]), int(r[0])) for r in narrow]
    seen, prev = set(), None
    for k in key:
        if k != prev:
            assert k not in seen
            seen.add(k)
            prev = k


def test_small_trees_get_no_wide_items_unless_asked():
    """A tree on which a warp of the streaming kernel would visit four page slots or fewer is left to that
    kernel alone (the second kernel's launch costs more than it saves); setting the threshold explicitly
    switches the exception off, and larger trees keep their wide items."""
    def items(name, wide=None):
        wl = make_workload(name)
        g = wl.geometry
        ctx = host_ctx(g.num_q_heads, g.num_kv_heads, g.head_dim, pages=1 << 15, max_path_entries=1 << 14)
        if wide is not None:
            ctx.set_option(ets.ETS_OPT_WIDE, wide)
        ctx.tree_build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node)
        n_narrow = ctx.get_stats()["n_narrow_items"]
        item = ctx.work_export()["item"]
        _check_work(ctx, wl.tree, wl.tree.tokens, g.num_kv_heads, g.gqa)
        return n_narrow, len(item)
    n_narrow, n_items = items("cfg2")
    assert n_narrow == n_items                  # root group of 64 rows, but only ~2.4 page slots per warp
    n_narrow, n_items = items("cfg2", wide=33)
    assert n_narrow < n_items
    n_narrow, n_items = items("cfg3_ets")
    assert n_narrow < n_items


def test_wide_limit_follows_the_kernel_that_would_end_last():
    """While ETS_OPT_WIDE is untouched the limit is 33 rows where the streaming kernel is on the critical path
    (little sharing: the width-256 tree) and 49 where the tcgen05 kernel would end last (most K/V under large
    query groups: the random-sharing tree, an ETS-pruned width-256 tree)."""
    def counts(name, wide=None):
        wl = make_workload(name)
        g = wl.geometry
        ctx = host_ctx(g.num_q_heads, g.num_kv_heads, g.head_dim, pages=1 << 16, max_path_tokens=1 << 16, max_path_entries=1 << 20, max_nodes=4096, max_leaves=1024)
        if wide is not None:
            ctx.set_option(ets.ETS_OPT_WIDE, wide)
        ctx.tree_build(wl.tree.parent, wl.tree.tokens, wl.tree.leaf_node)
        return ctx.get_stats()["n_narrow_items"], len(ctx.work_export()["item"])
    assert counts("cfg4") == counts("cfg4", wide=33) != counts("cfg4", wide=49)
    assert counts("cfg5c") == counts("cfg5c", wide=49) != counts("cfg5c", wide=33)
    assert counts("search_w256_ets") == counts("search_w256_ets", wide=49) != counts("search_w256_ets", wide=33)


def test_path_items_cover_every_path_once():
    """ETS_OPT_PATH_ITEMS: one item per (node that leaves sit at, kv head, tile of those leaves); its page slots
    are the node's whole path in root-to-node order; every leaf gets exactly one partial slot per kv head; the
    exported query groups are unchanged."""
    rng = np.random.default_rng(17)
    for _ in range(40):
        hkv = int(rng.choice([1, 2]))
        gqa = int(rng.choice([1, 4]))
        tree = random_small_tree(rng, max_nodes=10, max_tokens=60, max_leaves=6)
        # several query tokens per leaf node, as in a step prefill
        leaves = np.concatenate([np.full(int(rng.integers(1, 40)), n, np.int32) for n in sorted(set(tree.leaf_node.tolist()))])
        ctx = host_ctx(hq=hkv * gqa, hkv=hkv, max_leaves=leaves.shape[0], max_path_entries=leaves.shape[0] * 12,
                       max_path_tokens=1 << 12)
        ctx.tree_build(tree.parent, tree.tokens, leaves)
        groups = ctx.tree_export()["node_leaves"].copy()
        ctx.set_option(ets.ETS_OPT_PATH_ITEMS, 1)
        ctx.tree_build(tree.parent, tree.tokens, leaves)
        t, w = ctx.tree_export(), ctx.work_export()
        assert np.array_equal(t["node_leaves"], groups)
        seen = {}
        for it in w["item"]:
            ub, uc, head, lb, nl, slot0, seg, _ = (int(x) for x in it)
            assert seg == -1 and uc >= 1
            units = w["unit"][ub:ub + uc]
            node = int(units[-1][1])
            path = []
            v = node
            while v >= 0:
                path.append(v)
                v = int(tree.parent[v])
            expect = [(int(pg), n, 16 * j) for n in reversed(path)
                      for j, pg in enumerate(t["page_ids"][t["node_page_off"][n]:t["node_page_off"][n + 1]])]
            assert [(int(u[0]), int(u[1]), int(u[2])) for u in units] == expect
            for i in range(nl):
                seen.setdefault((slot0 + i, head), 0)
                seen[(slot0 + i, head)] += 1
        assert all(c == 1 for c in seen.values())
        for l in range(leaves.shape[0]):
            for h in range(hkv):
                k = l * hkv + h
                n_slots = w["leaf_slot_off"][k + 1] - w["leaf_slot_off"][k]
                has_pages = any(t["node_page_off"][n + 1] > t["node_page_off"][n] for n in _path(tree, int(leaves[l])))
                assert n_slots == (1 if has_pages else 0)


def _path(tree, node):
    out = []
    while node >= 0:
        out.append(node)
        node = int(tree.parent[node])
    return out


def test_rebuilding_the_current_tree_is_recognised_and_changes_nothing():
    """A rebuild with the same arrays, every node keeping its own pages, is a no-op; any difference (a capacity, a
    leaf, the keep list, an option) takes the ordinary path.  Either way the exported tables are what a fresh
    flatten of those arrays gives."""
    import time
    wl = make_workload("cfg4")
    t = wl.tree
    cap = t.tokens.copy()
    cap[t.leaf_node] += 20
    n, l, mpt, mpe, pages = bounds_for_tree(t.parent, cap + 16, t.leaf_node)
    cfg = ets.make_config(32, 8, 128, num_layers=2, max_nodes=n, max_leaves=l, max_path_tokens=mpt, max_path_entries=mpe,
                          pages_per_layer=pages + 64, device=-1)
    ctx = ets.EtsContext(cfg)
    keep = np.arange(t.n_nodes, dtype=np.int32)
    ctx.tree_build(t.parent, cap, t.leaf_node)
    first = ctx.tree_export()
    work = ctx.work_export()
    t0 = time.perf_counter()
    for _ in range(20):
        ctx.tree_build(t.parent, cap, t.leaf_node, keep_pages_of=keep)
    same = (time.perf_counter() - t0) / 20
    again = ctx.tree_export()
    for k in first:
        assert np.array_equal(first[k], again[k]), k
    assert np.array_equal(work["item"], ctx.work_export()["item"])
    # a changed capacity is a real rebuild (more pages for the leaves' nodes), and going back restores the tables
    cap2 = cap.copy()
    cap2[t.leaf_node] += 16
    t0 = time.perf_counter()
    ctx.tree_build(t.parent, cap2, t.leaf_node, keep_pages_of=keep)
    changed = time.perf_counter() - t0
    assert ctx.tree_export()["page_ids"].shape[0] > first["page_ids"].shape[0]
    assert same < changed
    # a different keep list is not the identity: pages are reassigned
    ctx.tree_build(t.parent, cap, t.leaf_node)
    ctx.tree_build(t.parent, cap, t.leaf_node, keep_pages_of=np.full(t.n_nodes, -1, np.int32))
    assert ctx.tree_export()["page_ids"].shape == first["page_ids"].shape


def test_new_entry_points_refuse_a_host_only_context_and_bad_arguments():
    """Every device entry point is refused on a context without a device, before anything is attempted; options
    outside their range are refused; the probes check their arguments before any launch."""
    ctx = host_ctx()
    ctx.tree_build([-1, 0], [4, 4], [1])
    for call in (lambda: ctx.decode_step_host_layers(0, 1, 1024, 1024),
                 lambda: ctx.decode_step(0, 1024, 1024, 1024, 1024),
                 lambda: ctx.tree_attn_decode_static(0, 1024, 1024)):
        with pytest.raises(ets.EtsError) as e:
            call()
        assert e.value.code == ets.ETS_ERR_STATE
    with pytest.raises(ets.EtsError) as e:
        ctx.decode_step_host_layers(0, 0, 1024, 1024)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG
    ctx.set_option(ets.ETS_OPT_LAUNCH_CHAIN, 0)
    ctx.set_option(ets.ETS_OPT_LAUNCH_CHAIN, 1)
    ctx.set_option(ets.ETS_OPT_TEST_FIRST_WAIT_POLLS, 0)
    ctx.set_option(ets.ETS_OPT_TEST_FIRST_WAIT_POLLS, -1)
    with pytest.raises(ets.EtsError) as e:
        ctx.set_option(ets.ETS_OPT_TEST_FIRST_WAIT_POLLS, 1 << 40)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG
    for args in ((0, 1 << 20, 8192, 2, 148, 0), (4096, 1 << 20, 1000, 2, 148, 4096), (4096, 1 << 20, 8192, 9, 148, 4096),
                 (4096, 1 << 20, 16384, 2, 148, 4096), (4096, 1 << 20, 8192, 2, 0, 4096)):
        with pytest.raises(ets.EtsError) as e:   # null buffer, odd chunk, depth, shared memory, grid
            ets.ets_probe_stream_read(*args)
        assert e.value.code == ets.ETS_ERR_INVALID_ARG
    with pytest.raises(ets.EtsError) as e:
        ets.ets_probe_empty_launch(0, 0, 4096)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG
