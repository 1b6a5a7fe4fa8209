"""Glue for the GPU parity tests: generator -> library (through the C ABI) and -> oracle."""
import numpy as np
import torch

import paper_2502_13575_b200 as ets
from paper_2502_13575_b200.runner import context_for_tree
from oracle.tree_attention import tree_decode_attention, bf16_bits_to_f64
from workloads import node_kv_bits, query_bits

ABS_TOL = 2e-3   # |gpu - oracle| <= 2e-3 + 1e-2 |oracle| on bf16 inputs with fp32 accumulation
REL_TOL = 1e-2


def bits_to_dev(bits: np.ndarray, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def node_values(tree, geom, value_seed, layer, lengths=None):
    lengths = tree.tokens if lengths is None else lengths
    ks, vs = [], []
    for n in range(tree.n_nodes):
        k, v = node_kv_bits(value_seed, n, int(lengths[n]), geom.num_kv_heads, geom.head_dim, layer)
        ks.append(k)
        vs.append(v)
    return ks, vs


def fill_layer(ctx, layer, ks, vs, nodes=None):
    nodes = list(range(len(ks))) if nodes is None else nodes
    nodes = [n for n in nodes if ks[n].shape[0] > 0]
    if not nodes:
        return
    k_all = bits_to_dev(np.concatenate([ks[n] for n in nodes], axis=0))
    v_all = bits_to_dev(np.concatenate([vs[n] for n in nodes], axis=0))
    ctx.kv_append(layer, nodes, [ks[n].shape[0] for n in nodes], k_all, v_all)


def check_close(gpu_bits, oracle, what=""):
    got = bf16_bits_to_f64(gpu_bits)
    err = np.abs(got - oracle)
    bound = ABS_TOL + REL_TOL * np.abs(oracle)
    worst = float((err - bound).max())
    assert worst <= 0, f"{what}: max excess over tolerance {worst:.3e}, max abs err {float(err.max()):.3e}"
    return float(err.max())


def run_and_check(tree, geom, value_seed, *, layers=(0,), qscale=1.0, chunk_pages=None, kernel=None, wide=None,
                  cap=None, lengths=None, leaves_subset=None, host_api=False, sm_scale=0.0, ctx=None,
                  aligned_q=False):
    """Build, fill, decode every requested layer, compare with the oracle.  Returns the context."""
    cap = tree.tokens if cap is None else cap
    lengths = tree.tokens if lengths is None else lengths
    n_layers = max(layers) + 1
    if ctx is None:
        ctx = context_for_tree(geom.num_q_heads, geom.num_kv_heads, geom.head_dim, tree.parent, cap,
                               tree.leaf_node, num_layers=n_layers, chunk_pages=chunk_pages,
                               sm_scale=sm_scale)
        if kernel is not None:
            ctx.set_option(ets.ETS_OPT_KERNEL, kernel)
        if wide is not None:
            ctx.set_option(ets.ETS_OPT_WIDE, wide)
        ctx.tree_build(tree.parent, cap, tree.leaf_node)
    L = tree.n_leaves
    for layer in layers:
        ks, vs = node_values(tree, geom, value_seed, layer, lengths)
        fill_layer(ctx, layer, ks, vs)
        qb = query_bits(value_seed, layer, L, geom.num_q_heads, geom.head_dim, qscale, aligned_with_node2=aligned_q)
        if host_api:
            q_h = torch.from_numpy(qb.view(np.int16)).pin_memory()
            out_h = torch.empty_like(q_h).pin_memory()
            lse_h = torch.empty((L, geom.num_q_heads), dtype=torch.float32).pin_memory()
            ctx.tree_attn_decode_host(layer, q_h, out_h, lse_h)
            torch.cuda.synchronize()
            out_bits = out_h.numpy().view(np.uint16)
            lse = lse_h.numpy().astype(np.float64)
        else:
            q = bits_to_dev(qb)
            out = torch.empty_like(q)
            lse_t = torch.empty((L, geom.num_q_heads), dtype=torch.float32, device="cuda")
            ctx.tree_attn_decode(layer, q, out, lse_t)
            torch.cuda.synchronize()
            out_bits = dev_to_bits(out)
            lse = lse_t.cpu().numpy().astype(np.float64)
        ctx.poll_status()
        ref, ref_lse = tree_decode_attention(tree.parent, lengths, tree.leaf_node, ks, vs, qb,
                                             geom.num_q_heads, geom.num_kv_heads,
                                             sm_scale=(sm_scale or None), leaves=leaves_subset)
        sel = slice(None) if leaves_subset is None else list(leaves_subset)
        check_close(out_bits[sel], ref[sel], f"layer {layer}")
        assert np.all(np.abs(lse[sel] - ref_lse[sel]) <= 1e-3 + 1e-3 * np.abs(ref_lse[sel])), "lse"
    return ctx
