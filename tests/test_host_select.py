"""The library's selection step (ets_select, host C++ branch and bound) against the enumeration oracle.
Runs without a GPU.  Equal optima may differ in which set is returned, so what is compared is what is
unique: the weights, the optimal value of Eq. 4, and that the returned set really has that value."""
import time

import numpy as np
import pytest

import paper_2502_13575_b200 as ets
from oracle.selection import rebase_weights, objective, select_brute, retained_nodes
from workloads import random_small_tree, make_workload


def _away_from_integers(reward, width, temperature, members=None):
    """True when no product N_i * share of Eq. 1 lies within 1e-9 of an integer, except the exact last one:
    then the ceilings cannot depend on the rounding of the sums."""
    idx = list(range(len(reward))) if members is None else list(members)
    order = sorted(idx, key=lambda i: (-reward[i], i))
    e = np.exp((np.array([reward[i] for i in order]) - reward[order[0]]) / temperature)
    left = width
    for k in range(len(order)):
        if left <= 0:
            break
        x = left * (e[k] / e[k:].sum())
        if k < len(order) - 1 and abs(x - round(x)) < 1e-9:
            return False
        left -= int(np.ceil(x))
    return True


@pytest.mark.parametrize("with_clusters", [False, True])
def test_small_trees_match_enumeration(with_clusters):
    rng = np.random.default_rng(11 + with_clusters)
    done = 0
    while done < 150:
        tree = random_small_tree(rng, max_nodes=12, max_leaves=9, allow_forest=bool(rng.integers(0, 2)))
        L = tree.n_leaves
        reward = rng.random(L)
        width = int(rng.integers(1, 33))
        temp = float(rng.choice([0.05, 0.2, 1.0]))
        lam_b = float(rng.choice([0.0, 0.2, 0.7, 1.5, 5.0]))
        lam_d = float(rng.choice([0.1, 0.5, 2.0])) if with_clusters else 0.0
        cl = rng.integers(-1, 4, size=L).astype(np.int32) if with_clusters else None
        if not _away_from_integers(reward, width, temp):
            continue
        got = ets.ets_select(tree.parent, tree.leaf_node, reward, cl, width=width, temperature=temp,
                             lambda_b=lam_b, lambda_d=lam_d)
        w = rebase_weights(reward, width, temp)
        assert got["weight"].tolist() == w.tolist()
        best, _ = select_brute(tree.parent, tree.leaf_node, w, cl, lam_b, lam_d)
        keep = [i for i in range(L) if got["keep"][i]]
        assert got["proven_optimal"] and len(keep) >= 1
        assert got["objective"] == pytest.approx(best, abs=1e-12)
        assert objective(tree.parent, tree.leaf_node, w, cl, keep, lam_b, lam_d) == pytest.approx(best, abs=1e-12)
        assert set(np.flatnonzero(got["node_kept"]).tolist()) == retained_nodes(tree.parent, tree.leaf_node, keep)
        assert got["n_kept"] == len(keep) and got["n_nodes_kept"] == int(got["node_kept"].sum())
        if _away_from_integers(reward, width, temp, keep):
            assert got["continuations"].tolist() == rebase_weights(reward, width, temp, members=keep).tolist()
        assert int(got["continuations"].sum()) == width and np.all(got["continuations"][got["keep"] == 0] == 0)
        done += 1


def test_arguments_are_checked():
    with pytest.raises(ets.EtsError) as e:
        ets.ets_select([-1, 0], [1], [0.5], width=0)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG
    with pytest.raises(ets.EtsError) as e:
        ets.ets_select([-1, 5], [1], [0.5], width=4)
    assert e.value.code == ets.ETS_ERR_BAD_TREE
    with pytest.raises(ets.EtsError) as e:
        ets.ets_select([-1, 0], [1], [float("nan")], width=4)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG
    with pytest.raises(ets.EtsError) as e:
        ets.ets_select([-1, 0], [1], [0.5], width=4, temperature=0.0)
    assert e.value.code == ets.ETS_ERR_INVALID_ARG


@pytest.mark.parametrize("name", ["cfg3_diverse", "cfg4"])
def test_search_width_trees(name):
    """Width 64 and 256: the exact search finishes, its value is at least that of the simple choices
    (keep everything weighted, keep the single best), the kept tree shrinks as lambda_b grows, and a large
    lambda_d covers every cluster."""
    tree = make_workload(name).tree
    rng = np.random.default_rng(3)
    L = tree.n_leaves
    reward = rng.random(L)
    cl = rng.integers(0, 12, size=L).astype(np.int32)
    sizes = []
    for lam_b in (0.0, 0.5, 1.0, 2.0):
        t0 = time.perf_counter()
        got = ets.ets_select(tree.parent, tree.leaf_node, reward, cl, width=L, temperature=0.2, lambda_b=lam_b, lambda_d=0.3)
        dt = time.perf_counter() - t0
        assert got["proven_optimal"] and dt < 5.0
        w = got["weight"]
        keep = np.flatnonzero(got["keep"]).tolist()
        assert objective(tree.parent, tree.leaf_node, w, cl, keep, lam_b, 0.3) == pytest.approx(got["objective"], abs=1e-10)
        everything = [i for i in range(L) if w[i] > 0]
        single = [int(np.argmax(w))]
        for other in (everything, single):
            assert got["objective"] >= objective(tree.parent, tree.leaf_node, w, cl, other, lam_b, 0.3) - 1e-10
        sizes.append(got["n_nodes_kept"])
    assert all(a >= b for a, b in zip(sizes, sizes[1:])) and sizes[-1] < sizes[0]
    got = ets.ets_select(tree.parent, tree.leaf_node, reward, cl, width=L, temperature=0.2, lambda_b=1.0, lambda_d=50.0)
    assert {int(cl[i]) for i in np.flatnonzero(got["keep"])} == set(cl.tolist())
