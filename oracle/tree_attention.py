"""Tree-decode attention by the definition, in fp64.  TEST INFRASTRUCTURE ONLY.

Setting (paper Section 4.1): a search tree of step nodes; a trajectory is a
root-to-leaf path; two trajectories that pass through the same node share that node's
KV cache.  A decode step issues one query per live leaf, and that query attends to all
KV tokens on the leaf's path (the paper's "KV cache state" of the trajectory,
Section 1).  With grouped-query attention, query head a reads KV head a // G where
G = num_q_heads // num_kv_heads (contiguous groups).

No mask and no positional transform are applied: the decode query is the newest token
and sees its whole path; rotary embedding, if any, happens before this step.

Inputs are bf16 bit patterns (uint16).  They are widened exactly to fp64; scores, the
max shift, exponentials, sums and the division are all fp64.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def leaf_path(parent: Sequence[int], node: int) -> List[int]:
    """Nodes from the root down to `node` (inclusive)."""
    path = []
    v = int(node)
    while v >= 0:
        path.append(v)
        v = int(parent[v])
    path.reverse()
    return path


def materialise_path(parent: Sequence[int], node_len: Sequence[int], leaf: int,
                     k_nodes: Sequence[np.ndarray], v_nodes: Sequence[np.ndarray]
                     ) -> Tuple[np.ndarray, np.ndarray]:
    """Concatenate, in root-to-leaf order, the first node_len[n] K and V rows of every
    node on the path.  Returns fp64 arrays [S, num_kv_heads, head_dim]."""
    ks, vs = [], []
    for n in leaf_path(parent, leaf):
        t = int(node_len[n])
        if t == 0:
            continue
        ks.append(bf16_bits_to_f64(k_nodes[n][:t]))
        vs.append(bf16_bits_to_f64(v_nodes[n][:t]))
    if not ks:
        raise ValueError("leaf path holds no KV tokens")
    return np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)


def tree_decode_attention(parent: Sequence[int], node_len: Sequence[int],
                          leaf_node: Sequence[int],
                          k_nodes: Sequence[np.ndarray], v_nodes: Sequence[np.ndarray],
                          q_bits: np.ndarray, num_q_heads: int, num_kv_heads: int,
                          sm_scale: Optional[float] = None,
                          leaves: Optional[Sequence[int]] = None
                          ) -> Tuple[np.ndarray, np.ndarray]:
    """out[l, a, :] = sum_t softmax_t(sm_scale * <q[l,a], K_l[t, a//G]>) * V_l[t, a//G]
    lse[l, a]    = log sum_t exp(sm_scale * <q[l,a], K_l[t, a//G]>)      (natural log)

    k_nodes[n], v_nodes[n]: uint16 [>= node_len[n], num_kv_heads, head_dim] per node.
    q_bits: uint16 [n_leaves, num_q_heads, head_dim].
    leaves: optional subset of leaf indices to evaluate (others are left as NaN).
    Returns (out fp64 [n_leaves, num_q_heads, head_dim], lse fp64 [n_leaves, num_q_heads]).
    """
    n_leaves = len(leaf_node)
    head_dim = int(q_bits.shape[-1])
    if num_q_heads % num_kv_heads:
        raise ValueError("num_q_heads must be a multiple of num_kv_heads")
    group = num_q_heads // num_kv_heads
    scale = (1.0 / math.sqrt(head_dim)) if sm_scale is None else float(sm_scale)
    q = bf16_bits_to_f64(q_bits)
    out = np.full((n_leaves, num_q_heads, head_dim), np.nan, dtype=np.float64)
    lse = np.full((n_leaves, num_q_heads), np.nan, dtype=np.float64)
    todo = range(n_leaves) if leaves is None else leaves
    for l in todo:
        k_path, v_path = materialise_path(parent, node_len, int(leaf_node[l]), k_nodes, v_nodes)
        for a in range(num_q_heads):
            h = a // group
            s = scale * (k_path[:, h, :] @ q[l, a, :])
            m = s.max()
            w = np.exp(s - m)
            z = w.sum()
            out[l, a, :] = (w @ v_path[:, h, :]) / z
            lse[l, a] = m + math.log(z)
    return out, lse


def tree_prefill_attention(parent: Sequence[int], node_len: Sequence[int], leaf_node: Sequence[int],
                           leaf_limit: Sequence[int],
                           k_nodes: Sequence[np.ndarray], v_nodes: Sequence[np.ndarray],
                           q_bits: np.ndarray, num_q_heads: int, num_kv_heads: int,
                           sm_scale: Optional[float] = None,
                           leaves: Optional[Sequence[int]] = None
                           ) -> Tuple[np.ndarray, np.ndarray]:
    """Attention of the tokens of a newly generated step (what the reward model and the prefill of a step
    compute; the paper scores every new step with a PRM, Section 5.1).  Every query is a "leaf" sitting at
    its step's node: it sees all tokens of the node's ancestors (their KV is shared, Section 4.1) and the
    first leaf_limit[l] tokens of its own node, i.e. the causal mask inside the step: the j-th of the T new
    tokens of a node that now holds `len` tokens has limit len - T + j + 1.  The paper prints no formula;
    this is textbook causal softmax attention over the trajectory, evaluated on the materialised sequence.
    With leaf_limit[l] = node_len[leaf_node[l]] it is tree_decode_attention."""
    n_leaves = len(leaf_node)
    head_dim = int(q_bits.shape[-1])
    group = num_q_heads // num_kv_heads
    scale = (1.0 / math.sqrt(head_dim)) if sm_scale is None else float(sm_scale)
    q = bf16_bits_to_f64(q_bits)
    out = np.full((n_leaves, num_q_heads, head_dim), np.nan, dtype=np.float64)
    lse = np.full((n_leaves, num_q_heads), np.nan, dtype=np.float64)
    for l in (range(n_leaves) if leaves is None else leaves):
        own = int(leaf_node[l])
        lim = int(leaf_limit[l])
        if not 0 <= lim <= int(node_len[own]):
            raise ValueError("leaf_limit must lie in [0, node_len of the leaf's node]")
        seen = list(node_len)
        seen[own] = lim                      # ancestors whole, own node up to the limit
        k_path, v_path = materialise_path(parent, seen, own, k_nodes, v_nodes)
        for a in range(num_q_heads):
            h = a // group
            s = scale * (k_path[:, h, :] @ q[l, a, :])
            m = s.max()
            w = np.exp(s - m)
            z = w.sum()
            out[l, a, :] = (w @ v_path[:, h, :]) / z
            lse[l, a] = m + math.log(z)
    return out, lse


def node_partial(k: np.ndarray, v: np.ndarray, q: np.ndarray, scale: float
                 ) -> Tuple[float, float, np.ndarray]:
    """Softmax partial of one query over one block of tokens: (m, l, o~) with
    m = max_t s_t, l = sum_t exp(s_t - m), o~ = sum_t exp(s_t - m) v_t.  An empty
    block gives (-inf, 0, 0)."""
    if k.shape[0] == 0:
        return -math.inf, 0.0, np.zeros(v.shape[-1], dtype=np.float64)
    s = scale * (k @ q)
    m = float(s.max())
    w = np.exp(s - m)
    return m, float(w.sum()), w @ v


def merge_partials(parts: Sequence[Tuple[float, float, np.ndarray]]) -> Tuple[np.ndarray, float]:
    """Combine partials of disjoint token blocks: with m* = max_j m_j,
    l* = sum_j l_j exp(m_j - m*), o = sum_j o~_j exp(m_j - m*) / l*, lse = m* + log l*.
    Empty partials (l_j = 0) are skipped.  This is the exact softmax of the union."""
    live = [p for p in parts if p[1] > 0.0]
    if not live:
        raise ValueError("all partials are empty")
    m_star = max(p[0] for p in live)
    l_star = 0.0
    acc = np.zeros_like(live[0][2])
    for m, l, o in live:
        w = math.exp(m - m_star)
        l_star += l * w
        acc = acc + o * w
    return acc / l_star, m_star + math.log(l_star)
