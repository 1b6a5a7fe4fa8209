"""Seeded bf16 K / V / Q values, addressable per (layer, node) and per (layer).

Values are N(0,1) float32 draws rounded to bf16 (round to nearest, ties to even) and
are handed around as uint16 bit patterns, since numpy has no bf16 type.

Addressing: node n's layer-0 K (or V) rows come from their own PCG64 stream seeded with
(value_seed, n, 0 or 1), drawn in [token, kv_head, dim] order, so the first T rows do
not depend on how many rows are drawn in total (a node that grows keeps its old rows).
Layer l > 0 re-uses the layer-0 rows with the feature axis rotated by l positions and
the sign flipped on odd layers: exact bf16 operations that a device can repeat on its
own copy, which keeps a 32-layer pool cheap to fill while every layer holds different
bytes.  Queries are drawn per layer from streams of their own: their seed key has a
fourth element, which no (value_seed, node, K|V) key of a node has.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

TOPOLOGY_SEED_BASE = 2502135750
VALUE_SEED_BASE = 2502135750 + 100


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even.  Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def layer_transform_bits(bits: np.ndarray, layer: int) -> np.ndarray:
    """Layer-0 rows -> layer-`layer` rows: rotate the last axis, flip sign on odd layers."""
    if layer == 0:
        return bits
    out = np.roll(bits, layer, axis=-1)
    if layer & 1:
        out = out ^ np.uint16(0x8000)
    return out


def _base_rows(value_seed: int, node: int, which: int, n_tokens: int, heads: int, dim: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([value_seed, node, which])))
    x = rng.standard_normal((n_tokens, heads, dim), dtype=np.float32)
    return f32_to_bf16_bits(x)


def node_kv_bits(value_seed: int, node: int, n_tokens: int, num_kv_heads: int, head_dim: int,
                 layer: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """K and V rows of one node in one layer: two uint16 arrays [n_tokens, num_kv_heads, head_dim]."""
    k = _base_rows(value_seed, node, 0, n_tokens, num_kv_heads, head_dim)
    v = _base_rows(value_seed, node, 1, n_tokens, num_kv_heads, head_dim)
    return layer_transform_bits(k, layer), layer_transform_bits(v, layer)


QUERY_STREAM_TAG = 0x51554552   # fourth element of a query stream's seed key


def query_bits(value_seed: int, layer: int, n_leaves: int, num_q_heads: int, head_dim: int,
               scale: float = 1.0, aligned_with_node2: bool = False) -> np.ndarray:
    """One decode query per leaf: uint16 [n_leaves, num_q_heads, head_dim].  `scale`
    multiplies the N(0,1) draw before rounding (peaked-softmax test cases use 4 and 8).

    `aligned_with_node2` draws from the key (value_seed, 2, layer) instead, which is also the key of
    node 2's K rows (layer 0) and V rows (layer 1): the query rows then repeat those rows bit for bit,
    every leaf below node 2 meets keys with score |q|^2/sqrt(d), and its softmax is sharply peaked.
    Kept as a deliberately hard case for the tests; no workload uses it."""
    key = [value_seed, 2, layer] if aligned_with_node2 else [value_seed, layer, 1, QUERY_STREAM_TAG]
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(key)))
    x = rng.standard_normal((n_leaves, num_q_heads, head_dim), dtype=np.float32)
    if scale != 1.0:
        x = x * np.float32(scale)
    return f32_to_bf16_bits(x)
