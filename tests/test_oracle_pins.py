"""Pins for the CPU oracle: each test ties it to something other than itself (a closed
form, a library routine, brute force, an invariant), so that a dropped term, a wrong
index or a swapped operand in oracle/ fails at least one of them."""
import math

import numpy as np
import pytest
import torch

from oracle import tree_attention as ota
from oracle.tree_attention import tree_decode_attention, node_partial, merge_partials, bf16_bits_to_f64
from workloads import random_small_tree, f32_to_bf16_bits, bf16_bits_to_f32
from _golden import read_golden


def _rand_bits(rng, shape, scale=1.0):
    return f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def _rand_tree_inputs(rng, tree, hq, hkv, d, qscale=1.0):
    k = [_rand_bits(rng, (int(t), hkv, d)) for t in tree.tokens]
    v = [_rand_bits(rng, (int(t), hkv, d)) for t in tree.tokens]
    q = _rand_bits(rng, (tree.n_leaves, hq, d), qscale)
    return k, v, q


def _nonempty(tree):
    """leaves whose path holds at least one token"""
    ok = []
    for l, node in enumerate(tree.leaf_node):
        s, v = 0, int(node)
        while v >= 0:
            s += int(tree.tokens[v])
            v = int(tree.parent[v])
        if s > 0:
            ok.append(l)
    return ok


# ---------------------------------------------------------------- bf16 widening
def test_bf16_widening_is_exact():
    # bit patterns with known values: 1.0, -2.0, 0.5, 3.140625 (0x4049), smallest normal
    bits = np.array([0x3F80, 0xC000, 0x3F00, 0x4049, 0x0080], dtype=np.uint16)
    want = [1.0, -2.0, 0.5, 3.140625, 2.0 ** -126]
    assert bf16_bits_to_f64(bits).tolist() == want
    # and against torch's own bf16 type
    t = torch.tensor([1.0, -2.0, 0.5, 3.140625, 0.1, -7.3e5], dtype=torch.float32).to(torch.bfloat16)
    tb = t.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bf16_bits_to_f64(tb), t.to(torch.float64).numpy())


# ---------------------------------------------------------------- P1 single token
def test_single_token_tree_returns_v_exactly():
    rng = np.random.default_rng(1)
    hq, hkv, d = 4, 2, 8
    k = [_rand_bits(rng, (1, hkv, d))]
    v = [_rand_bits(rng, (1, hkv, d))]
    q = _rand_bits(rng, (1, hq, d))
    out, lse = tree_decode_attention([-1], [1], [0], k, v, q, hq, hkv)
    for a in range(hq):
        h = a // (hq // hkv)
        assert np.array_equal(out[0, a], bf16_bits_to_f64(v[0][0, h]))
        want = float(np.dot(bf16_bits_to_f64(q[0, a]), bf16_bits_to_f64(k[0][0, h]))) / math.sqrt(d)
        assert lse[0, a] == pytest.approx(want, abs=1e-13)


# ---------------------------------------------------------------- P2 independent sequences
@pytest.mark.parametrize("hq,hkv,d", [(4, 1, 16), (8, 2, 32), (6, 3, 8)])
def test_leaves_split_at_root_equal_library_attention(hq, hkv, d):
    rng = np.random.default_rng(2)
    n_seq = 5
    lens = [int(x) for x in rng.integers(1, 40, size=n_seq)]
    # empty root, one private node per leaf
    parent = [-1] + [0] * n_seq
    tokens = [0] + lens
    leaves = list(range(1, n_seq + 1))
    k = [np.zeros((0, hkv, d), np.uint16)] + [_rand_bits(rng, (t, hkv, d)) for t in lens]
    v = [np.zeros((0, hkv, d), np.uint16)] + [_rand_bits(rng, (t, hkv, d)) for t in lens]
    q = _rand_bits(rng, (n_seq, hq, d))
    out, lse = tree_decode_attention(parent, tokens, leaves, k, v, q, hq, hkv)
    g = hq // hkv
    for i in range(n_seq):
        kt = torch.from_numpy(bf16_bits_to_f32(k[i + 1])).double()  # [T, hkv, d]
        vt = torch.from_numpy(bf16_bits_to_f32(v[i + 1])).double()
        qt = torch.from_numpy(bf16_bits_to_f32(q[i])).double()      # [hq, d]
        kt = kt.permute(1, 0, 2).repeat_interleave(g, dim=0)        # [hq, T, d]
        vt = vt.permute(1, 0, 2).repeat_interleave(g, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(qt[:, None, :], kt, vt)[:, 0, :]
        np.testing.assert_allclose(out[i], ref.numpy(), rtol=1e-12, atol=1e-13)
        ref_lse = torch.logsumexp((kt @ qt[:, :, None])[:, :, 0] / math.sqrt(d), dim=1)
        np.testing.assert_allclose(lse[i], ref_lse.numpy(), rtol=1e-12, atol=1e-13)


def test_prefill_of_a_root_step_is_causal_self_attention():
    """A step at the root (no ancestors) whose T tokens are all new: the prefill oracle must equal a
    library causal attention routine on that one sequence."""
    import torch
    from oracle.tree_attention import tree_prefill_attention
    rng = np.random.default_rng(61)
    hq, hkv, d, T = 4, 2, 8, 11
    g = hq // hkv
    k = [_rand_bits(rng, (T, hkv, d))]
    v = [_rand_bits(rng, (T, hkv, d))]
    q = _rand_bits(rng, (T, hq, d))
    out, lse = tree_prefill_attention([-1], [T], [0] * T, list(range(1, T + 1)), k, v, q, hq, hkv)
    kt = torch.from_numpy(bf16_bits_to_f32(k[0])).double().permute(1, 0, 2).repeat_interleave(g, dim=0)   # [hq, T, d]
    vt = torch.from_numpy(bf16_bits_to_f32(v[0])).double().permute(1, 0, 2).repeat_interleave(g, dim=0)
    qt = torch.from_numpy(bf16_bits_to_f32(q)).double().permute(1, 0, 2)                                  # [hq, T, d]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)                    # [hq, T, d]
    np.testing.assert_allclose(out, ref.permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-13)


def test_prefill_sees_ancestors_whole_and_own_step_causally():
    """Against the decode oracle: the query with limit t on node n equals a decode query on the tree in which
    n holds only its first t tokens; with the limit at the node's length it is the decode query itself; and
    (brute force) with an explicit mask over the concatenated path."""
    from oracle.tree_attention import tree_prefill_attention
    rng = np.random.default_rng(62)
    hq, hkv, d = 4, 2, 8
    done = 0
    while done < 25:
        tree = random_small_tree(rng, max_nodes=8, allow_forest=True, allow_empty_nodes=True)
        k, v, _ = _rand_tree_inputs(rng, tree, hq, hkv, d)
        leaf_nodes = [int(n) for n in tree.leaf_node if tree.tokens[n] > 0]
        if not leaf_nodes:
            continue
        leaves, limits = [], []
        for n in leaf_nodes:
            for t in sorted(set(int(x) for x in rng.integers(1, tree.tokens[n] + 1, size=2))):
                leaves.append(n)
                limits.append(t)
        q = _rand_bits(rng, (len(leaves), hq, d))
        out, lse = tree_prefill_attention(tree.parent, tree.tokens, leaves, limits, k, v, q, hq, hkv)
        for i, (n, t) in enumerate(zip(leaves, limits)):
            cut = tree.tokens.copy()
            cut[n] = t
            o1, l1 = tree_decode_attention(tree.parent, cut, [n], k, v, q[i:i + 1], hq, hkv)
            np.testing.assert_array_equal(out[i], o1[0])
            np.testing.assert_array_equal(lse[i], l1[0])
            # explicit mask over the whole path with the full node
            path = []
            x = n
            while x >= 0:
                path.append(x)
                x = int(tree.parent[x])
            path.reverse()
            kk = np.concatenate([bf16_bits_to_f32(k[p][:tree.tokens[p]]).astype(np.float64) for p in path])
            vv = np.concatenate([bf16_bits_to_f32(v[p][:tree.tokens[p]]).astype(np.float64) for p in path])
            visible = np.concatenate([np.ones(int(tree.tokens[p]), bool) if p != n else np.arange(int(tree.tokens[p])) < t
                                      for p in path])
            qq = bf16_bits_to_f32(q[i]).astype(np.float64)
            for a in range(hq):
                sc = (kk[:, a // (hq // hkv), :] @ qq[a]) / math.sqrt(d)
                wgt = np.where(visible, np.exp(sc), 0.0)
                np.testing.assert_allclose(out[i, a], (wgt @ vv[:, a // (hq // hkv), :]) / wgt.sum(), rtol=1e-11, atol=1e-12)
        full = [int(tree.tokens[n]) for n in leaf_nodes]
        qf = _rand_bits(rng, (len(leaf_nodes), hq, d))
        a1, b1 = tree_prefill_attention(tree.parent, tree.tokens, leaf_nodes, full, k, v, qf, hq, hkv)
        a2, b2 = tree_decode_attention(tree.parent, tree.tokens, leaf_nodes, k, v, qf, hq, hkv)
        np.testing.assert_array_equal(a1, a2)
        np.testing.assert_array_equal(b1, b2)
        done += 1


def test_forest_equals_its_trees_one_at_a_time():
    """Several problems in one call (a parent array with several roots) give, for every leaf, what the
    leaf's own tree gives alone: nothing couples the problems."""
    from workloads.trees import concat_trees
    rng = np.random.default_rng(44)
    hq, hkv, d = 4, 2, 8
    for _ in range(10):
        trees = [random_small_tree(rng, max_nodes=6, allow_forest=False, allow_empty_nodes=False) for _ in range(3)]
        parts = [_rand_tree_inputs(rng, t, hq, hkv, d) for t in trees]
        forest = concat_trees(trees)
        k = [x for p in parts for x in p[0]]
        v = [x for p in parts for x in p[1]]
        q = np.concatenate([p[2] for p in parts])
        out, lse = tree_decode_attention(forest.parent, forest.tokens, forest.leaf_node, k, v, q, hq, hkv)
        l0 = 0
        for t, (kk, vv, qq) in zip(trees, parts):
            o1, s1 = tree_decode_attention(t.parent, t.tokens, t.leaf_node, kk, vv, qq, hq, hkv)
            np.testing.assert_array_equal(out[l0:l0 + t.n_leaves], o1)
            np.testing.assert_array_equal(lse[l0:l0 + t.n_leaves], s1)
            l0 += t.n_leaves


# ---------------------------------------------------------------- P3 node splitting
def test_splitting_a_node_changes_nothing():
    rng = np.random.default_rng(3)
    hq, hkv, d = 4, 2, 8
    for _ in range(20):
        tree = random_small_tree(rng, allow_forest=False)
        k, v, q = _rand_tree_inputs(rng, tree, hq, hkv, d)
        live = _nonempty(tree)
        if not live:
            continue
        base, base_lse = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv, leaves=live)
        # split node s into (s: first t1 tokens) -> (new node: rest); children of s re-hang below the new node
        s = int(rng.integers(0, tree.n_nodes))
        t = int(tree.tokens[s])
        t1 = int(rng.integers(0, t + 1))
        n = tree.n_nodes
        # new numbering: old nodes 0..s stay, new node gets index s+1, old i>s -> i+1
        def remap(i):
            return i if i <= s else i + 1
        parent2 = [0] * (n + 1)
        tokens2 = [0] * (n + 1)
        k2 = [None] * (n + 1)
        v2 = [None] * (n + 1)
        for i in range(n):
            p = int(tree.parent[i])
            if p == s:
                p2 = s + 1
            else:
                p2 = remap(p) if p >= 0 else -1
            parent2[remap(i)] = p2
            tokens2[remap(i)] = int(tree.tokens[i])
            k2[remap(i)], v2[remap(i)] = k[i], v[i]
        parent2[s + 1] = s
        tokens2[s], tokens2[s + 1] = t1, t - t1
        k2[s], k2[s + 1] = k[s][:t1], k[s][t1:]
        v2[s], v2[s + 1] = v[s][:t1], v[s][t1:]
        leaves2 = [(s + 1) if int(x) == s else remap(int(x)) for x in tree.leaf_node]
        out2, lse2 = tree_decode_attention(parent2, tokens2, leaves2, k2, v2, q, hq, hkv, leaves=live)
        np.testing.assert_allclose(out2[live], base[live], rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse2[live], base_lse[live], rtol=0, atol=1e-12)


# ---------------------------------------------------------------- P4 brute force
def _brute_force(parent, tokens, leaf_node, k, v, q, hq, hkv, scale):
    """Triple loop in Python floats, explicit exp without a max shift."""
    kf = [bf16_bits_to_f32(x).astype(np.float64).tolist() for x in k]
    vf = [bf16_bits_to_f32(x).astype(np.float64).tolist() for x in v]
    qf = bf16_bits_to_f32(q).astype(np.float64).tolist()
    g = hq // hkv
    d = len(qf[0][0])
    out, lse = [], []
    for l, node in enumerate(leaf_node):
        chain = []
        x = int(node)
        while x != -1:
            chain.insert(0, x)
            x = int(parent[x])
        row_o, row_l = [], []
        for a in range(hq):
            h = a // g
            num = [0.0] * d
            den = 0.0
            for n in chain:
                for t in range(int(tokens[n])):
                    s = 0.0
                    for c in range(d):
                        s += qf[l][a][c] * kf[n][t][h][c]
                    e = math.exp(s * scale)
                    den += e
                    for c in range(d):
                        num[c] += e * vf[n][t][h][c]
            row_o.append([x / den for x in num])
            row_l.append(math.log(den))
        out.append(row_o)
        lse.append(row_l)
    return np.array(out), np.array(lse)


def test_brute_force_on_tiny_trees():
    rng = np.random.default_rng(4)
    hq, hkv, d = 4, 2, 4
    done = 0
    while done < 25:
        tree = random_small_tree(rng, max_nodes=6, max_tokens=4, max_leaves=4)
        live = _nonempty(tree)
        if len(live) != tree.n_leaves:
            continue
        k, v, q = _rand_tree_inputs(rng, tree, hq, hkv, d)
        out, lse = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv)
        bo, bl = _brute_force(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv, 1.0 / math.sqrt(d))
        np.testing.assert_allclose(out, bo, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(lse, bl, rtol=1e-12, atol=1e-13)
        done += 1


# ---------------------------------------------------------------- P5 closed forms
def test_zero_query_gives_mean_of_v_and_log_length():
    rng = np.random.default_rng(5)
    hq, hkv, d = 2, 1, 8
    tree = random_small_tree(rng, max_nodes=8, allow_empty_nodes=False)
    k, v, _ = _rand_tree_inputs(rng, tree, hq, hkv, d)
    q = np.zeros((tree.n_leaves, hq, d), np.uint16)
    out, lse = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv)
    for l, node in enumerate(tree.leaf_node):
        rows = []
        x = int(node)
        while x >= 0:
            rows.append(bf16_bits_to_f32(v[x]).astype(np.float64)[:, 0, :])
            x = int(tree.parent[x])
        allv = np.concatenate(rows)
        for a in range(hq):
            np.testing.assert_allclose(out[l, a], allv.mean(axis=0), rtol=1e-13, atol=1e-14)
            assert lse[l, a] == pytest.approx(math.log(allv.shape[0]), abs=1e-13)


def test_equal_keys_give_mean_of_v_with_shifted_lse():
    rng = np.random.default_rng(6)
    hq, hkv, d = 2, 2, 8
    krow = _rand_bits(rng, (1, hkv, d))
    tokens = [3, 5]
    k = [np.repeat(krow, t, axis=0) for t in tokens]
    v = [_rand_bits(rng, (t, hkv, d)) for t in tokens]
    q = _rand_bits(rng, (1, hq, d), 8.0)  # large scores: exp without a max shift would overflow in fp32
    out, lse = tree_decode_attention([-1, 0], tokens, [1], k, v, q, hq, hkv)
    for a in range(hq):
        allv = np.concatenate([bf16_bits_to_f32(x).astype(np.float64)[:, a, :] for x in v])
        np.testing.assert_allclose(out[0, a], allv.mean(axis=0), rtol=1e-13, atol=1e-14)
        s = float(np.dot(bf16_bits_to_f64(q[0, a]), bf16_bits_to_f64(krow[0, a]))) / math.sqrt(d)
        assert lse[0, a] == pytest.approx(s + math.log(8), abs=1e-12)


def test_powers_of_two_worked_example():
    g = read_golden("softmax_powers_of_two.txt")
    tokens = g["tokens"]
    d = 2
    karr = np.array(g["k"], dtype=np.float32).reshape(-1, 1, d)
    varr = np.array(g["v"], dtype=np.float32).reshape(-1, 1, d)
    # every listed value is exactly representable in bf16
    kb, vb = f32_to_bf16_bits(karr), f32_to_bf16_bits(varr)
    assert np.array_equal(bf16_bits_to_f32(kb), karr) and np.array_equal(bf16_bits_to_f32(vb), varr)
    ks, vs, o = [], [], 0
    for t in tokens:
        ks.append(kb[o:o + t])
        vs.append(vb[o:o + t])
        o += t
    q = f32_to_bf16_bits(np.array(g["q"], dtype=np.float32).reshape(1, 1, d))
    out, lse = tree_decode_attention(g["parent"], tokens, g["leaf_node"], ks, vs, q, 1, 1, sm_scale=math.log(2.0))
    want = np.array(g["out_num"], dtype=np.float64) / g["out_den"][0]
    np.testing.assert_allclose(out[0, 0], want, rtol=1e-14)
    assert lse[0, 0] == pytest.approx(math.log(g["lse_exp"][0]), abs=1e-14)


# ---------------------------------------------------------------- P6 permutation invariance
def test_token_and_sibling_order_do_not_matter():
    rng = np.random.default_rng(7)
    hq, hkv, d = 4, 2, 8
    tree = random_small_tree(rng, max_nodes=10, allow_forest=False, allow_empty_nodes=False)
    k, v, q = _rand_tree_inputs(rng, tree, hq, hkv, d)
    base, _ = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv)
    k2, v2 = [], []
    for kn, vn in zip(k, v):
        perm = rng.permutation(kn.shape[0])
        k2.append(kn[perm])
        v2.append(vn[perm])
    out2, _ = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k2, v2, q, hq, hkv)
    np.testing.assert_allclose(out2, base, rtol=0, atol=1e-13)
    # reorder the leaves: rows move with them
    perm = rng.permutation(tree.n_leaves)
    out3, _ = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node[perm], k, v, q[perm], hq, hkv)
    np.testing.assert_array_equal(out3, base[perm])


# ---------------------------------------------------------------- P7 convexity
def test_outputs_are_convex_combinations():
    rng = np.random.default_rng(8)
    hq, hkv, d = 4, 1, 8
    tree = random_small_tree(rng, max_nodes=10, allow_forest=False, allow_empty_nodes=False)
    k, v, q = _rand_tree_inputs(rng, tree, hq, hkv, d, qscale=4.0)
    out, _ = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv)
    for l, node in enumerate(tree.leaf_node):
        rows = []
        x = int(node)
        while x >= 0:
            rows.append(bf16_bits_to_f32(v[x]).astype(np.float64)[:, 0, :])
            x = int(tree.parent[x])
        allv = np.concatenate(rows)
        assert (out[l] <= allv.max(axis=0) + 1e-12).all()
        assert (out[l] >= allv.min(axis=0) - 1e-12).all()


# ---------------------------------------------------------------- P8 merge identity
@pytest.mark.parametrize("qscale", [1.0, 8.0])
def test_per_node_partials_merge_to_the_direct_result(qscale):
    rng = np.random.default_rng(9)
    hq, hkv, d = 4, 2, 16
    for _ in range(10):
        tree = random_small_tree(rng, max_nodes=8)
        live = _nonempty(tree)
        if not live:
            continue
        k, v, q = _rand_tree_inputs(rng, tree, hq, hkv, d, qscale)
        out, lse = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, k, v, q, hq, hkv, leaves=live)
        scale = 1.0 / math.sqrt(d)
        qf = bf16_bits_to_f64(q)
        for l in live:
            for a in range(hq):
                h = a // (hq // hkv)
                parts = []
                x = int(tree.leaf_node[l])
                while x >= 0:
                    parts.append(node_partial(bf16_bits_to_f64(k[x])[:, h, :], bf16_bits_to_f64(v[x])[:, h, :], qf[l, a], scale))
                    x = int(tree.parent[x])
                o, s = merge_partials(parts)
                np.testing.assert_allclose(o, out[l, a], rtol=1e-12, atol=1e-13)
                assert s == pytest.approx(lse[l, a], abs=1e-12)


# ---------------------------------------------------------------- P9 duplicate leaves
def test_duplicate_leaves():
    rng = np.random.default_rng(10)
    hq, hkv, d = 2, 1, 8
    parent, tokens = [-1, 0, 0], [3, 2, 4]
    k = [_rand_bits(rng, (t, hkv, d)) for t in tokens]
    v = [_rand_bits(rng, (t, hkv, d)) for t in tokens]
    q = _rand_bits(rng, (3, hq, d))
    q[1] = q[0]
    out, _ = tree_decode_attention(parent, tokens, [1, 1, 1], k, v, q, hq, hkv)
    assert np.array_equal(out[0], out[1])
    assert not np.array_equal(out[0], out[2])


# ---------------------------------------------------------------- errors
def test_empty_path_is_an_error():
    with pytest.raises(ValueError):
        tree_decode_attention([-1], [0], [0], [np.zeros((0, 1, 4), np.uint16)], [np.zeros((0, 1, 4), np.uint16)],
                              np.zeros((1, 1, 4), np.uint16), 1, 1)


# ---------------------------------------------------------------- planted mistakes are caught
def test_pins_catch_planted_mistakes(monkeypatch):
    """Plant three plausible mistakes in the oracle (on the CPU) and check a pin fails."""
    # (1) the scale is dropped
    monkeypatch.setattr(ota.math, "sqrt", lambda x: 1.0)
    with pytest.raises(AssertionError):
        test_leaves_split_at_root_equal_library_attention(4, 1, 16)
    monkeypatch.undo()
    # (2) the root is left off every path
    real = ota.leaf_path
    monkeypatch.setattr(ota, "leaf_path", lambda parent, node: real(parent, node)[1:] or real(parent, node))
    with pytest.raises(AssertionError):
        test_brute_force_on_tiny_trees()
    monkeypatch.undo()
    # (3) node lengths are ignored (whole buffers are read): growing buffers must not change the result
    rng = np.random.default_rng(11)
    k = [_rand_bits(rng, (6, 1, 4))]
    v = [_rand_bits(rng, (6, 1, 4))]
    q = _rand_bits(rng, (1, 1, 4))
    short, _ = tree_decode_attention([-1], [3], [0], k, v, q, 1, 1)
    exact, _ = tree_decode_attention([-1], [3], [0], [k[0][:3]], [v[0][:3]], q, 1, 1)
    assert np.array_equal(short, exact)
