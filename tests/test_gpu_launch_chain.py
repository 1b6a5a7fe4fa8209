"""The launch chain (ETS_OPT_LAUNCH_CHAIN: append -> streaming kernel -> tcgen05 kernel -> merge as programmatic
dependent launches on one stream) against ordinary launches, and the time-out path of the attention kernels."""
import numpy as np
import pytest
import torch

import paper_2502_13575_b200 as ets
from paper_2502_13575_b200.runner import context_for_tree
from workloads import make_workload, query_bits, node_kv_bits
from oracle.tree_attention import tree_decode_attention
from _harness import node_values, fill_layer, bits_to_dev, dev_to_bits, check_close, run_and_check

pytestmark = pytest.mark.gpu


def _filled_context(wl, layers, headroom, wide=None, chain=1, overlap=0):
    g, tree = wl.geometry, wl.tree
    cap = tree.tokens.copy()
    cap[tree.leaf_node] += headroom
    ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, cap, tree.leaf_node, num_layers=layers)
    ctx.set_option(ets.ETS_OPT_LAUNCH_CHAIN, chain)
    ctx.set_option(ets.ETS_OPT_OVERLAP_APPEND, overlap)
    if wide is not None:
        ctx.set_option(ets.ETS_OPT_WIDE, wide)
    ctx.tree_build(tree.parent, cap, tree.leaf_node)
    for l in range(layers):
        ks, vs = node_values(tree, g, wl.value_seed, l)
        fill_layer(ctx, l, ks, vs)
    return ctx


@pytest.mark.parametrize("name,wide", [("cfg2", 33), ("cfg2", 0), ("cfg5a", None), ("cfg3_ets", None)])
def test_chained_launches_give_the_bits_of_ordinary_launches(name, wide):
    """Many decode steps queued back to back without a synchronisation in between (so that the kernels of
    neighbouring calls really overlap where the chain lets them): the chained launches, with and without the
    append running under the preceding merge, produce exactly the outputs of ordinary launches, and the last
    step agrees with the oracle on every leaf."""
    wl = make_workload(name)
    g, tree = wl.geometry, wl.tree
    L, layers, T = tree.n_leaves, 3, 5
    newk = node_kv_bits(wl.value_seed + 77, 0, T * L, g.num_kv_heads, g.head_dim)
    nk = [bits_to_dev(np.ascontiguousarray(newk[0].reshape(T, L, g.num_kv_heads, g.head_dim)[t])) for t in range(T)]
    nv = [bits_to_dev(np.ascontiguousarray(newk[1].reshape(T, L, g.num_kv_heads, g.head_dim)[t])) for t in range(T)]
    qs = [[bits_to_dev(query_bits(wl.value_seed, 10 * t + l, L, g.num_q_heads, g.head_dim)) for l in range(layers)] for t in range(T)]
    results = {}
    for mode, (chain, overlap) in {"plain": (0, 0), "chain": (1, 0), "chain+overlap": (1, 1)}.items():
        ctx = _filled_context(wl, layers, T, wide=wide, chain=chain, overlap=overlap)
        outs = []
        for t in range(T):
            for l in range(layers):
                out = torch.empty_like(qs[t][l])
                lse = torch.empty((L, g.num_q_heads), dtype=torch.float32, device="cuda")
                ctx.decode_step(l, nk[t], nv[t], qs[t][l], out, lse)
                outs.append((out, lse))
        torch.cuda.synchronize()
        ctx.poll_status()
        results[mode] = [(dev_to_bits(o), s.cpu().numpy()) for o, s in outs]
        del ctx
    for mode in ("chain", "chain+overlap"):
        for i, ((a, la), (b, lb)) in enumerate(zip(results["plain"], results[mode])):
            assert np.array_equal(a, b) and np.array_equal(la, lb), (mode, i)
    # the last call (last token, last layer) against the oracle
    l = layers - 1
    ks, vs = node_values(tree, g, wl.value_seed, l)
    lengths = tree.tokens.copy()
    kk = newk[0].reshape(T, L, g.num_kv_heads, g.head_dim)
    vv = newk[1].reshape(T, L, g.num_kv_heads, g.head_dim)
    for i, n in enumerate(tree.leaf_node):
        ks[n] = np.concatenate([ks[n], kk[:, i]])
        vs[n] = np.concatenate([vs[n], vv[:, i]])
    lengths[tree.leaf_node] += T
    qb = query_bits(wl.value_seed, 10 * (T - 1) + l, L, g.num_q_heads, g.head_dim)
    ref, _ = tree_decode_attention(tree.parent, lengths, tree.leaf_node, ks, vs, qb, g.num_q_heads, g.num_kv_heads)
    check_close(results["chain+overlap"][-1][0], ref, name)


@pytest.mark.parametrize("wide", [0, 17])
def test_a_wait_that_runs_out_raises_the_status_and_leaves_the_context_usable(wide):
    """The first wait for data of every worker is told to give up at once (ETS_OPT_TEST_FIRST_WAIT_POLLS = 0): the
    workers take their time-out path (raise the status word, start nothing new, wait with the ordinary bound for
    the copies they had started, which do arrive, release tensor memory, return).  Nothing faults or hangs;
    ets_poll_status reports ETS_ERR_DEVICE_TIMEOUT once, and the next ordinary call on the same context, whose
    item queue the aborted launch must have rewound, is correct against the oracle."""
    wl = make_workload("cfg1")
    g, tree = wl.geometry, wl.tree
    ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, tree.tokens, tree.leaf_node)
    ctx.set_option(ets.ETS_OPT_WIDE, wide)      # 17: the root (8 leaves x 4 heads = 32 rows) goes to the tcgen05 kernel
    ctx.tree_build(tree.parent, tree.tokens, tree.leaf_node)
    st = ctx.get_stats()
    assert (st["n_items"] > st["n_narrow_items"]) == (wide > 0)
    ks, vs = node_values(tree, g, wl.value_seed, 0)
    fill_layer(ctx, 0, ks, vs)
    qb = query_bits(wl.value_seed, 0, tree.n_leaves, g.num_q_heads, g.head_dim)
    q = bits_to_dev(qb)
    out = torch.empty_like(q)
    ctx.set_option(ets.ETS_OPT_TEST_FIRST_WAIT_POLLS, 0)
    ctx.tree_attn_decode(0, q, out, None)
    torch.cuda.synchronize()
    with pytest.raises(ets.EtsError) as e:
        ctx.poll_status()
    assert e.value.code == ets.ETS_ERR_DEVICE_TIMEOUT
    ctx.poll_status()                            # the word was cleared by the read
    ctx.set_option(ets.ETS_OPT_TEST_FIRST_WAIT_POLLS, -1)
    for _ in range(2):
        out.fill_(float("nan"))
        ctx.tree_attn_decode(0, q, out, None)
        torch.cuda.synchronize()
        ctx.poll_status()
        ref, _ = tree_decode_attention(tree.parent, tree.tokens, tree.leaf_node, ks, vs, qb, g.num_q_heads, g.num_kv_heads)
        check_close(dev_to_bits(out), ref, "call after a timed-out launch")


@pytest.mark.parametrize("pipeline", [0, 1])
def test_layers_in_one_host_call_equal_one_host_call_per_layer(pipeline):
    """ets_decode_step_host_layers over eleven layers (groups of four, four and three through both staging areas,
    twice in a row) gives the bits and the lengths of one ets_decode_step_host per layer and of the device-pointer
    step, and agrees with the oracle on the last layer."""
    from workloads.loader import DecodeJob
    wl = make_workload("cfg2")
    g, tree = wl.geometry, wl.tree
    layers = 11
    jobs = {k: DecodeJob(wl, headroom=4, device=0, layers=layers, host_buffers=(k != "device")) for k in ("group", "single", "device")}
    for j in jobs.values():
        j.ctx.set_option(ets.ETS_OPT_HOST_PIPELINE, pipeline if j is not jobs["device"] else 0)
    for step in range(2):
        jobs["group"].step_host()
        jobs["single"].step_host_per_layer()
        jobs["device"].step()
        torch.cuda.synchronize()
        a = jobs["group"].out_h.numpy().view(np.uint16)
        b = jobs["single"].out_h.numpy().view(np.uint16)
        c = dev_to_bits(jobs["device"].out)
        assert np.array_equal(a, b) and np.array_equal(a, c), step
    for j in jobs.values():
        j.ctx.poll_status()
    for l in (0, 5, layers - 1):
        assert jobs["group"].ctx.get_node_len(l).tolist() == jobs["device"].ctx.get_node_len(l).tolist()
    leaves = list(range(tree.n_leaves))
    node_len, ks, vs = jobs["group"].oracle_inputs(layers - 1, leaves)
    ref, _ = tree_decode_attention(tree.parent, node_len, tree.leaf_node, ks, vs, jobs["group"].q_bits[layers - 1],
                                   g.num_q_heads, g.num_kv_heads)
    check_close(jobs["group"].out_h.numpy().view(np.uint16)[layers - 1], ref, "last layer through the grouped host call")
