"""Oracle for the ETS selection step (test infrastructure only; the library never imports this).

Plain, slow restatement of Section 4 and Appendix B of the paper in fp64:

  rebase_weights   Eq. 1 / Eq. 3: walk the trajectories from the highest reward down; trajectory i gets
                   W_i = ceil(N_i * exp(R_i / T_R) / sum_{k in A_i} exp(R_k / T_R)), where A_i are the
                   trajectories not served yet (i included) and N_i the continuations still to hand out.
                   The paper defers the update of N_i and A_i to the REBASE code it builds on; the reading
                   taken here: N_1 = width, N_{i+1} = N_i - W_i, A_{i+1} = A_i without i, and once N_i <= 0
                   the remaining trajectories get 0.
  objective        Eq. 4: sum_{i in S} W_i / sum_i W_i - lambda_b |V_S| / |V_A| + lambda_d |C_S| / |C_A|,
                   V_S = nodes with a selected leaf at or below them, V_A = all nodes of the tree, C_S =
                   clusters with a selected leaf.  (Eq. 6 prints the coverage constraint as z_k <= x_i for
                   every i in C_k, which would need all members kept; the prose says a cluster counts when
                   any member is kept, which is what Eq. 4 rewards: the prose is followed.)
  select_brute     the maximiser of Eq. 4 over all non-empty leaf subsets, by enumeration (small L only).
  ets_step         weights -> selection -> weights again over the kept trajectories (Eq. 3).

Pins: tests/test_oracle_selection.py (hand-worked trees, lambda = 0 and large-lambda closed forms,
monotonicity in lambda_b, invariance under relabelling; ets_step as a whole on a hand-worked six-node tree).
"""
from __future__ import annotations

import itertools
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np


def rebase_weights(reward: Sequence[float], width: int, temperature: float,
                   members: Optional[Sequence[int]] = None) -> np.ndarray:
    """Eq. 1 (all trajectories) or Eq. 3 (`members`: the retained ones).  Ties in reward keep index order."""
    n = len(reward)
    w = np.zeros(n, np.int64)
    idx = list(range(n)) if members is None else list(members)
    order = sorted(idx, key=lambda i: (-float(reward[i]), i))
    shift = max((float(reward[i]) for i in order), default=0.0)
    e = {i: math.exp((float(reward[i]) - shift) / temperature) for i in order}
    remaining = int(width)
    for pos, i in enumerate(order):
        if remaining <= 0:
            break
        denom = sum(e[k] for k in order[pos:])
        w[i] = math.ceil(remaining * (e[i] / denom))   # N_i times the share, as Eq. 1 is written: the last share is exactly 1
        remaining -= int(w[i])
    return w


def retained_nodes(parent: Sequence[int], leaf_node: Sequence[int], selected: Sequence[int]) -> set:
    keep = set()
    for i in selected:
        v = int(leaf_node[i])
        while v >= 0 and v not in keep:
            keep.add(v)
            v = int(parent[v])
    return keep


def objective(parent, leaf_node, weights, cluster, selected, lambda_b: float, lambda_d: float) -> float:
    total_w = float(sum(int(x) for x in weights))
    gain = sum(int(weights[i]) for i in selected) / total_w if total_w > 0 else 0.0
    cost = lambda_b * len(retained_nodes(parent, leaf_node, selected)) / len(parent)
    cover = 0.0
    if cluster is not None:
        all_c = {int(c) for c in cluster if int(c) >= 0}
        if all_c:
            cover = lambda_d * len({int(cluster[i]) for i in selected if int(cluster[i]) >= 0}) / len(all_c)
    return gain - cost + cover


def select_brute(parent, leaf_node, weights, cluster, lambda_b: float, lambda_d: float) -> Tuple[float, List[int]]:
    """Best non-empty subset by enumeration; among equal objectives the first in enumeration order."""
    n = len(leaf_node)
    if n > 16:
        raise ValueError("enumeration is for small cases")
    best, best_set = -math.inf, []
    for r in range(1, n + 1):
        for sub in itertools.combinations(range(n), r):
            val = objective(parent, leaf_node, weights, cluster, sub, lambda_b, lambda_d)
            if val > best + 1e-15:
                best, best_set = val, list(sub)
    return best, best_set


def ets_step(parent, leaf_node, reward, cluster, width: int, temperature: float, lambda_b: float, lambda_d: float):
    """One selection step: (weights W, kept leaves, continuations W' per leaf, objective value)."""
    w = rebase_weights(reward, width, temperature)
    val, keep = select_brute(parent, leaf_node, w, cluster, lambda_b, lambda_d)
    w2 = rebase_weights(reward, width, temperature, members=keep)
    return w, keep, w2, val
