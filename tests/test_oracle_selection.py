"""Pins for the selection oracle (oracle/selection.py): values worked by hand from Eq. 1 and Eq. 4 of the
paper, closed forms at the ends of the lambda range, and invariants."""
import math

import numpy as np
import pytest

from oracle.selection import rebase_weights, retained_nodes, objective, select_brute, ets_step
from workloads import random_small_tree


def test_rebase_weights_by_hand():
    # Eq. 1 with exp(R/T) = 3 and 1, five continuations: ceil(5 * 3/4) = 4, then ceil(1 * 1/1) = 1
    assert rebase_weights([math.log(3.0), 0.0], 5, 1.0).tolist() == [4, 1]
    # the order is by reward, not by index
    assert rebase_weights([0.0, math.log(3.0)], 5, 1.0).tolist() == [1, 4]
    # equal rewards: ceil(4/4), ceil(3/3), ceil(2/2), ceil(1/1)
    assert rebase_weights([0.5] * 4, 4, 0.2).tolist() == [1, 1, 1, 1]
    # exp = 4, 2, 1, 1 and 8 continuations: ceil(8*4/8)=4, ceil(4*2/4)=2, ceil(2*1/2)=1, ceil(1*1/1)=1
    r = [math.log(4.0), math.log(2.0), 0.0, 0.0]
    assert rebase_weights(r, 8, 1.0).tolist() == [4, 2, 1, 1]
    # the budget runs out before the list does: ceil(2*4/8)=1, ceil(1*2/4)=1, then nothing is left
    assert rebase_weights(r, 2, 1.0).tolist() == [1, 1, 0, 0]
    # Eq. 3: the same rule over the retained trajectories only
    assert rebase_weights(r, 8, 1.0, members=[1, 3]).tolist() == [0, 6, 0, 2]   # ceil(8*2/3)=6, ceil(2*1/1)=2


def test_rebase_weights_invariants():
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(1, 20))
        width = int(rng.integers(1, 64))
        r = rng.random(n)
        t = float(rng.choice([0.05, 0.2, 1.0, 10.0]))
        w = rebase_weights(r, width, t)
        assert int(w.sum()) == width and w.min() >= 0      # every share is at most what is left, the last takes the rest
        order = np.argsort(-r, kind="stable")
        served = w[order]
        assert np.all(served[np.argmax(served == 0):] == 0) or served.min() > 0   # zeros only at the tail
    # temperature limits: all to the best; nearly even shares, where the ceiling still favours the best
    # (3 * 0.3333334 rounds up to 2, then ceil(1 * 0.5000001) = 1 and nothing is left for the last)
    assert rebase_weights([0.1, 0.9, 0.5], 6, 1e-3).tolist() == [0, 6, 0]
    assert rebase_weights([0.1, 0.9, 0.5], 3, 1e6).tolist() == [0, 2, 1]


#      0
#     / \
#    1   2
#   / \   \
#  3   4   5      leaves 0..2 sit at nodes 3, 4, 5
PARENT = [-1, 0, 0, 1, 1, 2]
LEAVES = [3, 4, 5]


def test_objective_by_hand():
    w = [3, 1, 4]
    assert retained_nodes(PARENT, LEAVES, [0]) == {0, 1, 3}
    assert retained_nodes(PARENT, LEAVES, [0, 1]) == {0, 1, 3, 4}
    assert retained_nodes(PARENT, LEAVES, [0, 2]) == {0, 1, 2, 3, 5}
    # Eq. 4 without clusters: 3/8 - 0.6 * 3/6
    assert objective(PARENT, LEAVES, w, None, [0], 0.6, 0.0) == pytest.approx(3 / 8 - 0.3)
    # leaves 0 and 1 share nodes 0 and 1: (3+1)/8 - 0.6 * 4/6
    assert objective(PARENT, LEAVES, w, None, [0, 1], 0.6, 0.0) == pytest.approx(0.5 - 0.4)
    # with clusters {0,1} -> a, {2} -> b and lambda_d = 0.5: one of two clusters covered
    assert objective(PARENT, LEAVES, w, [7, 7, 9], [0, 1], 0.6, 0.5) == pytest.approx(0.5 - 0.4 + 0.25)
    # leaves 1 and 2 meet only at the root: five of six nodes, both clusters
    assert objective(PARENT, LEAVES, w, [7, 7, 9], [1, 2], 0.6, 0.5) == pytest.approx(5 / 8 - 0.5 + 0.5)
    # best subset by hand at lambda_b = 0.6, no clusters: {2} gives 0.5 - 0.3 = 0.2, {0} 0.075, {0,2} 0.875 - 0.5,
    # {0,1,2} 1 - 0.6 = 0.4, {0,2} = 0.375, {1,2} = 0.625 - 0.5: the full set wins
    val, keep = select_brute(PARENT, LEAVES, w, None, 0.6, 0.0)
    assert keep == [0, 1, 2] and val == pytest.approx(0.4)
    # at lambda_b = 1.2 the shares are {2}: 0.5 - 0.6 = -0.1, {0,1,2}: 1 - 1.2 = -0.2, {0,2}: 0.875 - 1.0
    val, keep = select_brute(PARENT, LEAVES, w, None, 1.2, 0.0)
    assert keep == [2] and val == pytest.approx(-0.1)


def test_ets_step_by_hand():
    """The whole step on the six-node tree, every value worked out from Eq. 1, Eq. 4 and Eq. 3.
    exp(R/T) = 5, 2, 6 and eight continuations (no product below lands on an integer, where the ceiling
    would hang on the last bit of exp).  Eq. 1: leaf 2 first, ceil(8*6/13) = ceil(3.69) = 4; then leaf 0,
    ceil(4*5/7) = ceil(2.86) = 3; then leaf 1, ceil(1*2/2) = 1."""
    r = [math.log(5.0), math.log(2.0), math.log(6.0)]
    # lambda_b = 1.2: {2} gives 4/8 - 1.2*3/6 = -0.1, the best (see test_objective_by_hand); Eq. 3 hands all
    # eight continuations to the one kept trajectory
    w, keep, w2, val = ets_step(PARENT, LEAVES, r, None, 8, 1.0, 1.2, 0.0)
    assert w.tolist() == [3, 1, 4] and keep == [2] and w2.tolist() == [0, 0, 8] and val == pytest.approx(-0.1)
    # lambda_b = 0.9: {0,2}: 7/8 - 0.9*5/6 = 0.125; {0,1,2}: 1 - 0.9 = 0.1; {2}: 0.5 - 0.45 = 0.05; {1,2}: 5/8 - 0.75 < 0;
    # {0}: 3/8 - 0.45 < 0; {1}: 1/8 - 0.45 < 0; {0,1}: 0.5 - 0.6 < 0.  Eq. 3 over {0, 2}: leaf 2 gets
    # ceil(8*6/11) = ceil(4.36) = 5, leaf 0 ceil(3*5/5) = 3; the pruned leaf gets nothing
    w, keep, w2, val = ets_step(PARENT, LEAVES, r, None, 8, 1.0, 0.9, 0.0)
    assert w.tolist() == [3, 1, 4] and keep == [0, 2] and w2.tolist() == [3, 0, 5] and val == pytest.approx(0.125)
    # clusters {0,1} and {2}, lambda_b = 1.2, lambda_d = 0.5: {0,2}: 7/8 - 1 + 0.5 = 0.375; {0,1,2}: 1 - 1.2 + 0.5 = 0.3;
    # {2}: -0.1 + 0.25 = 0.15; {1,2}: 5/8 - 1 + 0.5 = 0.125; {0}: 3/8 - 0.6 + 0.25 = 0.025; {0,1}: 0.5 - 0.8 + 0.25 < 0;
    # {1}: 1/8 - 0.6 + 0.25 < 0
    w, keep, w2, val = ets_step(PARENT, LEAVES, r, [7, 7, 9], 8, 1.0, 1.2, 0.5)
    assert keep == [0, 2] and w2.tolist() == [3, 0, 5] and val == pytest.approx(0.375)
    # a colder temperature changes Eq. 1 and with it the choice: T = 0.5 squares the ratios (25, 4, 36):
    # ceil(8*36/65) = ceil(4.43) = 5, ceil(3*25/29) = ceil(2.59) = 3, nothing left for leaf 1; at lambda_b = 0.9:
    # {0,2}: 8/8 - 0.75 = 0.25 wins over {2}: 5/8 - 0.45 and {0,1,2}: 1 - 0.9; Eq. 3: ceil(8*36/61) = 5, then 3
    w, keep, w2, val = ets_step(PARENT, LEAVES, r, None, 8, 0.5, 0.9, 0.0)
    assert w.tolist() == [3, 0, 5] and keep == [0, 2] and w2.tolist() == [3, 0, 5] and val == pytest.approx(0.25)


def test_lambda_zero_keeps_every_weighted_leaf_and_large_lambda_keeps_one():
    rng = np.random.default_rng(5)
    for _ in range(30):
        tree = random_small_tree(rng, max_nodes=9, max_leaves=7, allow_forest=False)
        L = tree.n_leaves
        w = rng.integers(0, 5, size=L)
        if w.sum() == 0:
            continue
        val, keep = select_brute(tree.parent, tree.leaf_node, w, None, 0.0, 0.0)
        assert val == pytest.approx(1.0) and set(i for i in range(L) if w[i] > 0) <= set(keep)
        val, keep = select_brute(tree.parent, tree.leaf_node, w, None, 1e6, 0.0)
        depth = [len(retained_nodes(tree.parent, tree.leaf_node, [i])) for i in range(L)]
        assert len(retained_nodes(tree.parent, tree.leaf_node, keep)) == min(depth)


def test_retained_tree_shrinks_as_lambda_b_grows_and_coverage_term_covers():
    rng = np.random.default_rng(6)
    for _ in range(20):
        tree = random_small_tree(rng, max_nodes=10, max_leaves=8, allow_forest=False)
        L = tree.n_leaves
        w = rng.integers(1, 6, size=L)
        sizes = []
        for lam in (0.0, 0.3, 0.8, 1.5, 4.0):
            _, keep = select_brute(tree.parent, tree.leaf_node, w, None, lam, 0.0)
            sizes.append(len(retained_nodes(tree.parent, tree.leaf_node, keep)))
        assert all(a >= b for a, b in zip(sizes, sizes[1:]))
        cl = rng.integers(0, 3, size=L)
        _, keep = select_brute(tree.parent, tree.leaf_node, w, cl, 0.5, 100.0)
        assert {int(cl[i]) for i in keep} == {int(c) for c in cl}


def test_relabelling_leaves_changes_nothing():
    rng = np.random.default_rng(7)
    tree = random_small_tree(rng, max_nodes=10, max_leaves=8, allow_forest=False)
    L = tree.n_leaves
    r = rng.random(L)
    cl = rng.integers(0, 3, size=L)
    w, keep, w2, val = ets_step(tree.parent, tree.leaf_node, r, cl, 16, 0.2, 0.7, 0.3)
    perm = rng.permutation(L)
    _, keep_p, w2_p, val_p = ets_step(tree.parent, tree.leaf_node[perm], r[perm], cl[perm], 16, 0.2, 0.7, 0.3)
    assert val_p == pytest.approx(val)
    assert int(w2_p.sum()) == int(w2.sum()) == 16
