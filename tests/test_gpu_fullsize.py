"""Full-size parity in the launch configuration bench.py times: the width-256, 32-layer workload
driven through workloads.loader.DecodeJob.step (flatten + append + decode per layer), checked
on sampled leaves and layers that the oracle computes one by one; plus properties that hold at
any size (finite outputs, convexity bounds are covered by the sampled comparison)."""
import numpy as np
import pytest
import torch

from workloads import make_workload
from workloads.loader import DecodeJob
from oracle.tree_attention import tree_decode_attention
from _harness import check_close, dev_to_bits

pytestmark = pytest.mark.gpu


def _check_job(job, layers, leaves):
    wl = job.wl
    g, tree = wl.geometry, wl.tree
    for layer in layers:
        node_len, ks, vs = job.oracle_inputs(layer, leaves)
        ref, _ = tree_decode_attention(tree.parent, node_len, tree.leaf_node, ks, vs, job.q_bits[layer],
                                       g.num_q_heads, g.num_kv_heads, leaves=leaves)
        got = dev_to_bits(job.out[layer])
        check_close(got[leaves], ref[leaves], f"{wl.name} layer {layer}")
    assert torch.isfinite(job.out.float()).all()


def test_cfg4_all_layers_sampled():
    wl = make_workload("cfg4")
    job = DecodeJob(wl, headroom=4, device=0, host_buffers=False)
    for _ in range(2):
        job.step()
    torch.cuda.synchronize()
    job.ctx.poll_status()
    rng = np.random.default_rng(3)
    leaves = sorted(set([0, wl.tree.n_leaves - 1] + [int(x) for x in rng.integers(0, wl.tree.n_leaves, 4)]))
    _check_job(job, [0, 13, 31], leaves)
    st = job.ctx.get_stats()
    assert st["unique_tokens"] == int(wl.tree.tokens.sum()) + 2 * wl.tree.n_leaves
    # the host-buffer entry points give the same bytes as the device ones
    job2 = DecodeJob(wl, headroom=4, device=0, layers=2, host_buffers=True)
    job2.step_host()
    torch.cuda.synchronize()
    ref_job = DecodeJob(wl, headroom=4, device=0, layers=2, host_buffers=False)
    ref_job.step()
    torch.cuda.synchronize()
    a = job2.out_h.view(torch.int16)[:2].numpy()
    b = ref_job.out.view(torch.int16).cpu().numpy()
    assert np.array_equal(a, b)


@pytest.mark.parametrize("name", ["cfg3_diverse", "cfg3_ets", "cfg5a", "cfg5c"])
def test_other_configs_through_the_step_path(name):
    wl = make_workload(name)
    job = DecodeJob(wl, headroom=3, device=0, host_buffers=False)
    job.step()
    torch.cuda.synchronize()
    job.ctx.poll_status()
    L = wl.tree.n_leaves
    _check_job(job, [0], [0, L // 3, L - 1])
