"""The search-built workloads (workloads/search.py): the multi-step bookkeeping with the library's selection step
(ets_select) against the same search driven by the enumeration oracle, the KV-size figures of ets_select, and the
shape of the width-64 / width-256 pairs.  Runs without a GPU."""
import numpy as np
import pytest

import paper_2502_13575_b200 as ets
from oracle.selection import ets_step, retained_nodes
from workloads import make_workload, run_search, SEARCH_NAMES
from workloads.search import library_select


def _oracle_select(lambda_b, lambda_d, temperature):
    def select(parent, leaf_node, reward, cluster, width):
        _, _, cont, _ = ets_step(parent, leaf_node, reward, cluster if lambda_d > 0 else None, width, temperature,
                                 lambda_b, lambda_d)
        return cont
    return select


@pytest.mark.parametrize("lambda_b,lambda_d", [(0.0, 0.0), (0.8, 0.0), (1.5, 0.4), (3.0, 0.2)])
def test_search_with_the_library_equals_search_with_the_oracle(lambda_b, lambda_d):
    """Width 7, five steps: at every step the library's continuations (branch and bound) must be the oracle's
    (enumeration), else the two searches part ways; so the final trees, the per-step KV sizes and the whole
    selection history agree.  (Equal optima could be broken differently: the draws are continuous, ties do not occur.)"""
    for seed in range(6):
        kw = dict(width=7, steps=5, root_tokens=40, len_lo=5, len_hi=30, seed=900 + seed, keep_history=True)
        a = run_search(library_select(lambda_b, lambda_d, 0.3), **kw)
        b = run_search(_oracle_select(lambda_b, lambda_d, 0.3), **kw)
        assert a.kv_tokens_per_step == b.kv_tokens_per_step and a.kept_per_step == b.kept_per_step
        assert np.array_equal(a.tree.parent, b.tree.parent) and np.array_equal(a.tree.tokens, b.tree.tokens)
        assert np.array_equal(a.tree.leaf_node, b.tree.leaf_node)
        for ha, hb in zip(a.history, b.history):
            assert np.array_equal(ha["continuations"], hb["continuations"])


def test_search_bookkeeping_invariants():
    tr = run_search(library_select(1.0, 0.3), width=9, steps=6, root_tokens=64, len_lo=8, len_hi=24, seed=5, keep_history=True)
    t = tr.tree
    assert t.n_leaves == 9 and tr.live_per_step == [9] * 6 and len(tr.kv_tokens_per_step) == 6
    assert np.all(t.parent[1:] < np.arange(1, t.n_nodes)) and t.parent[0] == -1
    # every node of the snapshot has a live trajectory below it; the last step's KV size is the snapshot's
    assert retained_nodes(t.parent, t.leaf_node, range(t.n_leaves)) == set(range(t.n_nodes))
    assert tr.kv_tokens_per_step[-1] == int(t.tokens.sum())
    # a selection step hands out exactly the width and the next step has that many leaves below the kept ones
    for h in tr.history:
        assert int(h["continuations"].sum()) == 9
    # pruning harder keeps fewer trajectories per step and a smaller search
    soft = run_search(library_select(0.0, 0.0), width=9, steps=6, root_tokens=64, len_lo=8, len_hi=24, seed=5)
    hard = run_search(library_select(4.0, 0.0), width=9, steps=6, root_tokens=64, len_lo=8, len_hi=24, seed=5)
    assert hard.kv_size < soft.kv_size and sum(hard.kept_per_step) < sum(soft.kept_per_step)


def test_kv_size_of_a_selection_step():
    #      0(10)
    #     /    \
    #   1(20)  2(30)
    #   /  \      \
    # 3(1) 4(2)   5(4)     leaves at 3, 4, 5; node 6 hangs below nothing live
    parent = [-1, 0, 0, 1, 1, 2, 2]
    tokens = [10, 20, 30, 1, 2, 4, 1000]
    got = ets.ets_select(parent, [3, 4, 5], [0.9, 0.8, 0.1], width=4, temperature=0.2, lambda_b=1.3, node_tokens=tokens)
    kept = set(np.flatnonzero(got["node_kept"]).tolist())
    assert got["kv_tokens_all"] == 10 + 20 + 30 + 1 + 2 + 4                      # node 6 has no trajectory below it
    assert got["kv_tokens_kept"] == sum(tokens[v] for v in kept)
    assert kept == retained_nodes(parent, [3, 4, 5], np.flatnonzero(got["keep"]).tolist())
    # without the table the figures stay zero
    got = ets.ets_select(parent, [3, 4, 5], [0.9, 0.8, 0.1], width=4, temperature=0.2, lambda_b=1.3)
    assert got["kv_tokens_kept"] == 0 and got["kv_tokens_all"] == 0


@pytest.mark.parametrize("stem,lo,hi", [("search_w64", 1.5, 1.75), ("search_w256", 1.7, 1.95)])
def test_search_pairs_reproduce_the_papers_kv_ratio(stem, lo, hi):
    """Table 1 / Table 2 of the paper: ETS shrinks the KV size of the search 1.5-1.7x at width 64 and 1.8x at
    width 256 against REBASE; the seeded pairs are tuned into those ranges."""
    base, pruned = make_workload(stem + "_rebase"), make_workload(stem + "_ets")
    width = 64 if stem == "search_w64" else 256
    assert base.tree.n_leaves == pruned.tree.n_leaves == width
    assert lo <= pruned.notes["kv_ratio_vs_rebase"] <= hi
    assert pruned.tree.tokens.sum() < base.tree.tokens.sum()
    assert set(SEARCH_NAMES) >= {stem + "_rebase", stem + "_ets"}
