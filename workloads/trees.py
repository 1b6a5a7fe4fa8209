"""Seeded search-tree topologies shaped like the paper's workloads.

The paper searches with widths 16 / 64 / 256 (Section 5.1, Table 1) over trees of
reasoning steps in which trajectories that share a node share its KV cache
(Section 4.1).  Its datasets and models are not available offline, so these
generators draw trees with the same shape parameters: a prompt node at the
root, a fixed number of search steps, a fixed number of live leaves, step
lengths of tens to ~150 tokens, and a controllable amount of prefix sharing
(the 1.8x KV-size ratio of Table 2 is reproduced by the cfg3 pair).

A tree is three int32 arrays:
  parent[i]    index of node i's parent, -1 for a root, always < i
  tokens[i]    number of KV tokens node i holds (T_n)
  leaf_node[l] the node at which live leaf l sits
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

from .values import TOPOLOGY_SEED_BASE, VALUE_SEED_BASE


@dataclass(frozen=True)
class Geometry:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int = 16
    num_layers: int = 1

    @property
    def gqa(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:
        # K and V, bf16, all KV heads, one layer
        return 2 * self.num_kv_heads * self.head_dim * 2


@dataclass
class Tree:
    parent: np.ndarray
    tokens: np.ndarray
    leaf_node: np.ndarray

    @property
    def n_nodes(self) -> int:
        return int(self.parent.shape[0])

    @property
    def n_leaves(self) -> int:
        return int(self.leaf_node.shape[0])


@dataclass
class Workload:
    name: str
    config_id: int
    geometry: Geometry
    tree: Tree
    value_seed: int
    topology_seed: int
    notes: Dict[str, float] = field(default_factory=dict)


CONFIG_NAMES = (
    "cfg1",
    "cfg2",
    "cfg3_diverse",
    "cfg3_ets",
    "cfg4",
    "cfg5a",
    "cfg5b",
    "cfg5c",
    "forest_w16x8",
    "forest_w64x8",
)

_GEOM = {
    1: Geometry(4, 1, 64, 16, 1),
    2: Geometry(32, 8, 128, 16, 1),
    3: Geometry(32, 8, 128, 16, 1),
    4: Geometry(32, 8, 128, 16, 32),
    5: Geometry(64, 8, 128, 16, 1),
}


def _as_tree(parent: List[int], tokens: List[int], leaves: List[int]) -> Tree:
    return Tree(
        np.asarray(parent, dtype=np.int32),
        np.asarray(tokens, dtype=np.int32),
        np.asarray(leaves, dtype=np.int32),
    )


def _drop_dead_and_renumber(parent: List[int], tokens: List[int], live: List[int]) -> Tree:
    """Keep only nodes with a live leaf below them; renumber breadth-first."""
    n = len(parent)
    alive = [False] * n
    for leaf in live:
        v = leaf
        while v >= 0 and not alive[v]:
            alive[v] = True
            v = parent[v]
    children: List[List[int]] = [[] for _ in range(n)]
    roots = []
    for i in range(n):
        if not alive[i]:
            continue
        if parent[i] < 0:
            roots.append(i)
        else:
            children[parent[i]].append(i)
    order: List[int] = []
    queue = list(roots)
    head = 0
    while head < len(queue):
        v = queue[head]
        head += 1
        order.append(v)
        queue.extend(children[v])
    new_id = {old: new for new, old in enumerate(order)}
    new_parent = [(-1 if parent[old] < 0 else new_id[parent[old]]) for old in order]
    new_tokens = [tokens[old] for old in order]
    new_leaves = sorted(new_id[leaf] for leaf in live)
    return _as_tree(new_parent, new_tokens, new_leaves)


def _branch_and_prune(seed: int, root_tokens: int, steps: int, width: int,
                      len_lo: int, len_hi: int) -> Tuple[Tree, int]:
    """Every live leaf draws 1-4 children per step; levels above `width` are cut back
    to `width` by a seeded choice without replacement.  Retries with seed + 1000*attempt
    until the last level has exactly `width` leaves."""
    attempt = 0
    while True:
        rng = np.random.Generator(np.random.PCG64(seed + 1000 * attempt))
        parent = [-1]
        tokens = [root_tokens]
        live = [0]
        for _ in range(steps):
            cand: List[int] = []
            for leaf in live:
                c = int(rng.integers(1, 5))
                for _k in range(c):
                    parent.append(leaf)
                    tokens.append(int(rng.integers(len_lo, len_hi + 1)))
                    cand.append(len(parent) - 1)
            if len(cand) > width:
                keep = np.sort(rng.choice(len(cand), size=width, replace=False))
                cand = [cand[int(i)] for i in keep]
            live = cand
        if len(live) == width:
            return _drop_dead_and_renumber(parent, tokens, live), attempt
        attempt += 1
        if attempt > 64:
            raise RuntimeError("branch-and-prune generator did not reach the width")


def _keep_fraction(seed: int, root_tokens: int, steps: int, width: int, keep: int,
                   len_lo: int, len_hi: int) -> Tree:
    """Step 1: root -> `width` children.  Each later step keeps `keep` of the current
    leaves (seeded) and spreads `width` children over them as evenly as possible."""
    rng = np.random.Generator(np.random.PCG64(seed))
    parent = [-1]
    tokens = [root_tokens]
    live = []
    for _ in range(width):
        parent.append(0)
        tokens.append(int(rng.integers(len_lo, len_hi + 1)))
        live.append(len(parent) - 1)
    for _ in range(steps - 1):
        kept_idx = np.sort(rng.choice(len(live), size=keep, replace=False))
        kept = [live[int(i)] for i in kept_idx]
        base = width // keep
        extra = width - base * keep
        counts = [base] * keep
        if extra:
            for i in rng.choice(keep, size=extra, replace=False):
                counts[int(i)] += 1
        nxt: List[int] = []
        for node, c in zip(kept, counts):
            for _k in range(c):
                parent.append(node)
                tokens.append(int(rng.integers(len_lo, len_hi + 1)))
                nxt.append(len(parent) - 1)
        live = nxt
    return _drop_dead_and_renumber(parent, tokens, live)


def concat_trees(trees: List[Tree]) -> Tree:
    """Several independent problems as one forest: node and leaf lists are concatenated, parents shifted."""
    parent, tokens, leaves, off = [], [], [], 0
    for t in trees:
        parent.append(np.where(t.parent >= 0, t.parent + off, -1))
        tokens.append(t.tokens)
        leaves.append(t.leaf_node + off)
        off += t.n_nodes
    return Tree(np.concatenate(parent).astype(np.int32), np.concatenate(tokens).astype(np.int32),
                np.concatenate(leaves).astype(np.int32))


def _unique_tokens(tree: Tree) -> int:
    return int(tree.tokens.astype(np.int64).sum())


def _cfg1() -> Tree:
    parent = [-1]
    tokens = [32]
    level = [0]
    for _ in range(3):
        nxt = []
        for p in level:
            for _k in range(2):
                parent.append(p)
                tokens.append(16)
                nxt.append(len(parent) - 1)
        level = nxt
    return _as_tree(parent, tokens, level)


def _cfg5a() -> Tree:
    parent = [-1]
    tokens = [1024]
    for _ in range(5):
        parent.append(len(parent) - 1)
        tokens.append(128)
    tip = len(parent) - 1
    leaves = []
    for _ in range(128):
        parent.append(tip)
        tokens.append(128)
        leaves.append(len(parent) - 1)
    return _as_tree(parent, tokens, leaves)


def _cfg5b() -> Tree:
    parent = [-1]
    tokens = [1024]
    tips = []
    for _ in range(128):
        parent.append(0)
        tokens.append(128)
        tips.append(len(parent) - 1)
    for _ in range(5):
        nxt = []
        for t in tips:
            parent.append(t)
            tokens.append(128)
            nxt.append(len(parent) - 1)
        tips = nxt
    return _as_tree(parent, tokens, tips)


_CACHE: Dict[str, Workload] = {}


def make_workload(name: str) -> Workload:
    """Build one of CONFIG_NAMES.  Deterministic; results are cached per process."""
    if name in _CACHE:
        return _CACHE[name]
    if name.startswith("search_"):
        from .search import make_search_workload   # grown by a seeded search whose selection step is the library's
        return make_search_workload(name)
    notes: Dict[str, float] = {}
    if name == "cfg1":
        cid, variant, tree = 1, 0, _cfg1()
    elif name == "cfg2":
        cid, variant = 2, 0
        tree, attempt = _branch_and_prune(TOPOLOGY_SEED_BASE + cid, 256, 4, 16, 64, 128)
        notes["attempt"] = attempt
    elif name in ("cfg3_diverse", "cfg3_ets"):
        cid = 3
        div_seed = TOPOLOGY_SEED_BASE + cid
        ets_seed = TOPOLOGY_SEED_BASE + cid + 10
        diverse = _keep_fraction(div_seed, 512, 8, 64, 56, 64, 128)
        u_div = _unique_tokens(diverse)
        if name == "cfg3_diverse":
            variant, tree = 0, diverse
            notes["keep"] = 56
        else:
            variant = 1
            best = None
            for k in range(1, 64):
                cand = _keep_fraction(ets_seed, 512, 8, 64, k, 64, 128)
                ratio = u_div / _unique_tokens(cand)
                if best is None or abs(ratio - 1.8) < abs(best[0] - 1.8):
                    best = (ratio, k, cand)
            ratio, k, tree = best
            notes["keep"] = k
            notes["kv_ratio_vs_diverse"] = ratio
    elif name == "cfg4":
        cid, variant = 4, 0
        tree, attempt = _branch_and_prune(TOPOLOGY_SEED_BASE + cid, 512, 12, 256, 96, 160)
        notes["attempt"] = attempt
    elif name == "cfg5a":
        cid, variant, tree = 5, 0, _cfg5a()
    elif name == "cfg5b":
        cid, variant, tree = 5, 1, _cfg5b()
    elif name == "cfg5c":
        cid, variant = 5, 2
        tree, attempt = _branch_and_prune(TOPOLOGY_SEED_BASE + cid + 20, 1024, 6, 128, 128, 128)
        notes["attempt"] = attempt
    elif name == "forest_w16x8":
        # eight concurrent problems (the paper serves 4 to 32 at a time, Section 5.3), each a width-16
        # tree drawn like cfg2 with its own seed; one parent array with eight roots
        cid, variant = 2, 5
        tree = concat_trees([_branch_and_prune(TOPOLOGY_SEED_BASE + cid + 10 * variant + 100 * (i + 1), 256, 4, 16, 64, 128)[0]
                             for i in range(8)])
        notes["problems"] = 8
    elif name == "forest_w64x8":
        # eight concurrent width-64 problems, each drawn like the ETS-like tree of cfg3 (keep 36 of 64)
        cid, variant = 3, 5
        tree = concat_trees([_keep_fraction(TOPOLOGY_SEED_BASE + cid + 10 * variant + 100 * (i + 1), 512, 8, 64, 36, 64, 128)
                             for i in range(8)])
        notes["problems"] = 8
    else:
        raise KeyError(f"unknown workload {name!r}; choose from {CONFIG_NAMES}")
    wl = Workload(
        name=name,
        config_id=cid,
        geometry=_GEOM[cid],
        tree=tree,
        value_seed=VALUE_SEED_BASE + cid + 1000 * variant,
        topology_seed=TOPOLOGY_SEED_BASE + cid + 10 * variant,
        notes=notes,
    )
    _CACHE[name] = wl
    return wl


def random_small_tree(rng: np.random.Generator, max_nodes: int = 12, max_tokens: int = 40,
                      max_leaves: int = 6, allow_forest: bool = True,
                      allow_empty_nodes: bool = True) -> Tree:
    """A small arbitrary tree (or forest) for property tests: parents precede children,
    leaves may repeat and may sit on internal nodes, nodes may hold zero tokens."""
    n = int(rng.integers(1, max_nodes + 1))
    parent = [-1]
    for i in range(1, n):
        lo = -1 if allow_forest and rng.random() < 0.15 else 0
        parent.append(int(rng.integers(lo, i)))
    lo_tok = 0 if allow_empty_nodes else 1
    tokens = [int(rng.integers(lo_tok, max_tokens + 1)) for _ in range(n)]
    n_leaves = int(rng.integers(1, max_leaves + 1))
    leaves = [int(rng.integers(0, n)) for _ in range(n_leaves)]
    return _as_tree(parent, tokens, leaves)


def tree_stats(tree: Tree) -> Dict[str, int]:
    """Counts used in reports: unique tokens U, and the token total a kernel without
    prefix sharing would read (the sum over leaves of their path lengths)."""
    depth_tokens = np.zeros(tree.n_nodes, dtype=np.int64)
    depth_nodes = np.zeros(tree.n_nodes, dtype=np.int64)
    for i in range(tree.n_nodes):
        p = int(tree.parent[i])
        depth_tokens[i] = int(tree.tokens[i]) + (depth_tokens[p] if p >= 0 else 0)
        depth_nodes[i] = 1 + (depth_nodes[p] if p >= 0 else 0)
    return {
        "n_nodes": tree.n_nodes,
        "n_leaves": tree.n_leaves,
        "unique_tokens": _unique_tokens(tree),
        "path_tokens": int(depth_tokens[tree.leaf_node].sum()),
        "path_nodes": int(depth_nodes[tree.leaf_node].sum()),
        "max_depth": int(depth_nodes[tree.leaf_node].max()) if tree.n_leaves else 0,
    }
