"""Full-size parity in the launch configuration bench.py times: every workload driven through
workloads.loader.DecodeJob.step (flatten + append + decode per layer) and compared with the oracle on
EVERY leaf: all 256 leaves of the width-256 tree on its first, a middle and its last layer, all leaves
of layer 0 for the others.  A defect tied to a single work item (a tail piece, a re-read tile) touches
a few rows only; sampling a handful of leaves would let it through."""
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


def test_cfg4_every_leaf_on_three_layers():
    wl = make_workload("cfg4")
    job = DecodeJob(wl, headroom=4, device=0, host_buffers=False)
    for _ in range(2):
        job.step()
    torch.cuda.synchronize()
    job.ctx.poll_status()
    _check_job(job, [0, 13, 31], list(range(wl.tree.n_leaves)))
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


@pytest.mark.parametrize("name", ["cfg3_diverse", "cfg3_ets", "cfg5a", "cfg5b", "cfg5c", "forest_w64x8",
                                  "search_w64_rebase", "search_w64_ets"])
def test_other_configs_through_the_step_path(name):
    wl = make_workload(name)
    job = DecodeJob(wl, headroom=3, device=0, layers=1, host_buffers=False)
    job.step()
    torch.cuda.synchronize()
    job.ctx.poll_status()
    _check_job(job, [0], list(range(wl.tree.n_leaves)))
