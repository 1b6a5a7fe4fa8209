"""Reference tree flattener: the canonical tables for a search tree.  TEST INFRASTRUCTURE ONLY.

The paper fixes the semantics, not a table format: a node is retained iff some retained
trajectory passes through it, and trajectories through a node share its KV (Section 4.1,
Appendix B); serving systems keep shared KV segments once and reference them (Section 2.2).
The table format below is this project's; what makes it checkable bit for bit are the
following rules, which the library's host flattener must obey as well.

Validity
  parent[i] in [-1, i): parents precede children; -1 marks a root; forests are allowed.
  cap_tokens[i] >= 0.  leaf_node[l] in [0, N); leaves may repeat and may sit on
  internal nodes.  Nodes with no leaf below them are legal.

Pages
  Page ids 0 .. pages_per_layer-1 live in a min-heap free list.  A build first returns
  to the heap every page that no node of the new tree keeps, then walks the new nodes in
  index order; a node takes ceil(cap_tokens / page_size) pages: first the pages it keeps
  from keep_pages_of[i] (a node index of the previous build, or -1), truncated to what it
  needs, then the lowest free ids in ascending order.  keep_pages_of must not name the
  same old node twice.  A kept node's token length carries over (clipped to the new cap);
  other nodes start at length 0.

Ordering
  node_leaves lists, per node, the leaves whose path contains it, ascending leaf index.
  leaf_path lists, per leaf, its path root first.  leaf_path_pos gives, per path entry,
  the leaf's position inside that node's node_leaves list.  All offsets are int32 CSR with
  a trailing total.
"""
from __future__ import annotations

import heapq
from typing import Dict, List, Optional, Sequence

import numpy as np


class BadTree(ValueError):
    pass


class PoolExhausted(RuntimeError):
    pass


class ReferenceFlattener:
    def __init__(self, page_size: int, pages_per_layer: int):
        self.page_size = int(page_size)
        self.free: List[int] = list(range(int(pages_per_layer)))
        heapq.heapify(self.free)
        self.node_pages: List[List[int]] = []
        self.node_len: List[int] = []
        self.cap: List[int] = []
        self.parent: List[int] = []

    def build(self, parent: Sequence[int], cap_tokens: Sequence[int],
              leaf_node: Sequence[int],
              keep_pages_of: Optional[Sequence[int]] = None) -> Dict[str, np.ndarray]:
        n = len(parent)
        n_prev = len(self.node_pages)
        if len(cap_tokens) != n:
            raise BadTree("cap_tokens length")
        for i in range(n):
            if not (-1 <= int(parent[i]) < i):
                raise BadTree(f"parent[{i}]")
            if int(cap_tokens[i]) < 0:
                raise BadTree(f"cap_tokens[{i}]")
        for l, node in enumerate(leaf_node):
            if not (0 <= int(node) < n):
                raise BadTree(f"leaf_node[{l}]")
        keep = [-1] * n if keep_pages_of is None else [int(x) for x in keep_pages_of]
        seen = set()
        for i, old in enumerate(keep):
            if old == -1:
                continue
            if not (0 <= old < n_prev) or old in seen:
                raise BadTree(f"keep_pages_of[{i}]")
            seen.add(old)

        need = [-(-int(c) // self.page_size) for c in cap_tokens]
        # work on copies so that a failure leaves the previous state untouched
        free = list(self.free)
        kept_pages: List[List[int]] = [[] for _ in range(n)]
        new_len = [0] * n
        claimed_old = [0] * n_prev  # pages of each old node that survive
        for i, old in enumerate(keep):
            if old >= 0:
                kept_pages[i] = self.node_pages[old][: need[i]]
                claimed_old[old] = len(kept_pages[i])
                new_len[i] = min(self.node_len[old], int(cap_tokens[i]))
        for old in range(n_prev):
            for pid in self.node_pages[old][claimed_old[old]:]:
                heapq.heappush(free, pid)
        pages: List[List[int]] = []
        for i in range(n):
            mine = list(kept_pages[i])
            while len(mine) < need[i]:
                if not free:
                    raise PoolExhausted(f"node {i}")
                mine.append(heapq.heappop(free))
            pages.append(mine)

        self.free = free
        self.node_pages = pages
        self.node_len = new_len
        self.cap = [int(c) for c in cap_tokens]
        self.parent = [int(p) for p in parent]

        depth = [0] * n
        for i in range(n):
            depth[i] = 0 if parent[i] < 0 else depth[parent[i]] + 1

        groups: List[List[int]] = [[] for _ in range(n)]
        paths: List[List[int]] = []
        path_pos: List[List[int]] = []
        for l, node in enumerate(leaf_node):
            path = []
            v = int(node)
            while v >= 0:
                path.append(v)
                v = int(parent[v])
            path.reverse()
            paths.append(path)
            # leaves are visited in ascending index, so each group list stays ascending
            # and the leaf's position in it is the list's length before the append
            path_pos.append([len(groups[v]) for v in path])
            for v in path:
                groups[v].append(l)

        return {
            "node_page_off": _csr_off(pages),
            "page_ids": _csr_val(pages),
            "node_leaf_off": _csr_off(groups),
            "node_leaves": _csr_val(groups),
            "leaf_path_off": _csr_off(paths),
            "leaf_path": _csr_val(paths),
            "leaf_path_pos": _csr_val(path_pos),
            "node_depth": np.asarray(depth, dtype=np.int32),
            "node_len": np.asarray(new_len, dtype=np.int32),
        }

    def append(self, node: int, n_new: int) -> int:
        """Grow a node's length; returns the old length.  Must stay within the cap."""
        if not (0 <= node < len(self.node_len)) or n_new < 0:
            raise BadTree("append arguments")
        old = self.node_len[node]
        if old + n_new > self.cap[node]:
            raise PoolExhausted("append beyond cap_tokens")
        self.node_len[node] = old + n_new
        return old


def _csr_off(rows) -> np.ndarray:
    off = np.zeros(len(rows) + 1, dtype=np.int64)
    for i, r in enumerate(rows):
        off[i + 1] = off[i] + len(r)
    return off.astype(np.int32)


def _csr_val(rows) -> np.ndarray:
    flat = [x for r in rows for x in r]
    return np.asarray(flat, dtype=np.int32)
