#!/usr/bin/env python
"""Benchmark of tree-decode attention over prefix-shared KV.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

A step is one pass of the whole path over the workload's tree: tree flatten (all pages kept),
then for each layer the append of one new token per leaf and tree-decode attention for every
leaf.  The metric is leaf-queries/s = leaves / (time of one step over all layers), summed over
GPUs (independent replicas, no collective).  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "tree_decode_attention_leaf_queries_per_s"
UNIT = "leaf-queries/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (0 = its own)")
    ap.add_argument("--chunk-pages", type=int, default=None)
    ap.add_argument("--kernel", type=int, default=None)
    ap.add_argument("--wide", type=int, default=None, help="0: no tcgen05 wide-group items")
    ap.add_argument("--chain", type=int, default=None, help="0: ordinary launches instead of the programmatic-dependent chain")
    ap.add_argument("--loop-tokens", type=int, default=16,
                    help="decode iterations of the search-step loop figure (0 = skip it)")
    ap.add_argument("--prefill", action="store_true",
                    help="time step-prefill attention (all tokens of the workload's last search step as queries) "
                         "instead of the decode step; prints its own JSON line")
    ap.add_argument("--segment-items", action="store_true",
                    help="with --prefill: the decode work decomposition (items per segment) instead of path items")
    ap.add_argument("--repeats", type=int, default=5, help="times the K-step timed loop is repeated (median reported)")
    ap.add_argument("--no-table", action="store_true", help="skip the per-workload table and the probes of the default run")
    ap.add_argument("--table-only", action="store_true", help="only the per-workload table and the probes")
    ap.add_argument("--table-workloads", default="", help="comma-separated subset of the table's workloads (with --table-only)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU time budget of the oracle sample")
    return ap.parse_args()


def workload_description(wl, layers):
    from workloads import tree_stats
    g, st = wl.geometry, tree_stats(wl.tree)
    return {
        "workload": wl.name,
        "tree": f"{st['n_leaves']} leaves, {st['n_nodes']} nodes, {st['unique_tokens']} unique tokens, "
                f"{st['path_tokens']} path tokens",
        "heads": f"{g.num_q_heads}q/{g.num_kv_heads}kv x {g.head_dim}",
        "layers": layers,
        "page_size": g.page_size,
        "topology_seed": wl.topology_seed,
        "value_seed": wl.value_seed,
    }


# ----------------------------------------------------------------------------- oracle timing
# The oracle is timed as it stands.  Its unit of work is one leaf (all query heads of one layer): the leaf's
# whole path is materialised and softmax attention is evaluated per head in fp64.  Leaves are independent, so
# the all-cores figure runs them on a pool of worker processes, one BLAS thread each, and `cores` is the number
# of workers that really ran; the one-core figure runs the same leaves in one process with one BLAS thread.
_ORACLE = {}


def _oracle_worker_init(path):
    """Worker start-up: one BLAS thread, K/V of the sampled paths mapped from the file the parent wrote."""
    try:
        from threadpoolctl import threadpool_limits
        _ORACLE["limit"] = threadpool_limits(limits=1)
    except Exception:
        pass
    meta = np.load(os.path.join(path, "meta.npz"))
    k_all = np.load(os.path.join(path, "k.npy"), mmap_mode="r")
    v_all = np.load(os.path.join(path, "v.npy"), mmap_mode="r")
    off = meta["off"]
    n_nodes = int(meta["parent"].shape[0])
    _ORACLE.update(parent=meta["parent"], tokens=meta["tokens"], leaf_node=meta["leaf_node"], q=meta["q"],
                   hq=int(meta["heads"][0]), hkv=int(meta["heads"][1]),
                   k=[k_all[off[n]:off[n + 1]] for n in range(n_nodes)],
                   v=[v_all[off[n]:off[n + 1]] for n in range(n_nodes)])


def _oracle_worker_leaf(leaf):
    """One leaf of one layer through the oracle; returns the seconds it took (-1.0: start-up probe)."""
    if leaf < 0:
        return -1.0
    from oracle.tree_attention import tree_decode_attention
    o = _ORACLE
    t0 = time.perf_counter()
    tree_decode_attention(o["parent"], o["tokens"], o["leaf_node"], o["k"], o["v"], o["q"], o["hq"], o["hkv"],
                          leaves=[int(leaf)])
    return time.perf_counter() - t0


def _oracle_sample_files(wl, leaves, path):
    """K/V of every node on the sampled leaves' paths (layer 0), written where the workers can map them."""
    from workloads import node_kv_bits, query_bits
    tree, g = wl.tree, wl.geometry
    need = set()
    for l in leaves:
        v = int(tree.leaf_node[l])
        while v >= 0 and v not in need:
            need.add(v)
            v = int(tree.parent[v])
    off = np.zeros(tree.n_nodes + 1, np.int64)
    ks, vs = [], []
    for n in range(tree.n_nodes):
        t = int(tree.tokens[n]) if n in need else 0
        off[n + 1] = off[n] + t
        if t:
            k, v = node_kv_bits(wl.value_seed, n, t, g.num_kv_heads, g.head_dim, 0)
            ks.append(k)
            vs.append(v)
    np.save(os.path.join(path, "k.npy"), np.concatenate(ks))
    np.save(os.path.join(path, "v.npy"), np.concatenate(vs))
    tokens = np.where(np.isin(np.arange(tree.n_nodes), list(need)), tree.tokens, 0).astype(np.int64)
    np.savez(os.path.join(path, "meta.npz"), parent=np.asarray(tree.parent), tokens=tokens,
             leaf_node=np.asarray(tree.leaf_node), off=off,
             q=query_bits(wl.value_seed, 0, tree.n_leaves, g.num_q_heads, g.head_dim),
             heads=np.array([g.num_q_heads, g.num_kv_heads]))


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_sample(wl, layers, budget_s, workers=None):
    """Time the oracle, as it stands, on a bounded sample of whole leaves of layer 0: first on one core, then on
    a pool of `workers` processes (default: every core this process may use).  Returns a dict with
    leaf-queries/s of a full step over `layers` layers for both, the worker count and a description."""
    import multiprocessing as mp
    import shutil
    tree = wl.tree
    workers = workers or host_cores()
    order = [int(x) for x in np.random.default_rng(0).permutation(tree.n_leaves)]
    # enough leaves to keep every worker busy for the budget; the paths' K/V is generated outside the timed part
    n_sample = min(tree.n_leaves, max(2 * workers, 8))
    sample = order[:n_sample]
    tmp = tempfile.mkdtemp(prefix="ets_oracle_")
    try:
        _oracle_sample_files(wl, sample, tmp)
        # ---- one core
        _oracle_worker_init(tmp)
        one_budget = max(1.0, 0.3 * budget_s)
        spent1, done1 = 0.0, 0
        for l in sample:
            spent1 += _oracle_worker_leaf(l)
            done1 += 1
            if spent1 >= one_budget:
                break
        lim = _ORACLE.pop("limit", None)
        if lim is not None:
            lim.restore_original_limits()
        per_leaf_1 = spent1 / done1
        # ---- all cores: a spawned pool (a fork after CUDA start-up would hang), warmed up before the clock starts
        ctx = mp.get_context("spawn")
        with ctx.Pool(workers, initializer=_oracle_worker_init, initargs=(tmp,)) as pool:
            pool.map(_oracle_worker_leaf, [-1] * (4 * workers))
            # about 0.7 of the budget if the workers scaled perfectly; at least every sampled leaf once
            n_jobs = max(n_sample, int(0.7 * budget_s * workers / max(per_leaf_1, 1e-4)))
            jobs = [sample[i % n_sample] for i in range(n_jobs)]
            t0 = time.perf_counter()
            pool.map(_oracle_worker_leaf, jobs, chunksize=1)
            wall = time.perf_counter() - t0
        per_leaf_all = wall / len(jobs)
    finally:
        shutil.rmtree(tmp, ignore_errors=True)
    return {
        "value": 1.0 / (per_leaf_all * layers), "value_one_core": 1.0 / (per_leaf_1 * layers), "cores": workers,
        "sample": (f"{len(jobs)} leaf evaluations ({n_sample} distinct leaves of {tree.n_leaves}) of {wl.name}, layer 0 only, "
                   f"on {workers} worker processes with one BLAS thread each ({wall:.1f} s wall); one core: {done1} leaves "
                   f"in {spent1:.1f} s; a full step is {layers} layers x {tree.n_leaves} leaves, scaled linearly"),
        "seconds": wall + spent1,
    }


def run_reference(args):
    """The reference arm: the fp64 CPU oracle timed on the host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from workloads import make_workload
    wl = make_workload(args.workload)
    layers = args.layers or wl.geometry.num_layers
    per_step_budget = max(1.0, min(8.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, ones = [], []
    res = None
    for i in range(args.warmup + args.steps):
        res = oracle_sample(wl, layers, per_step_budget)
        if i >= args.warmup:
            vals.append(res["value"])
            ones.append(res["value_one_core"])
    value = len(vals) / sum(1.0 / v for v in vals)
    ms = 1000.0 * wl.tree.n_leaves / value
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_description(wl, layers),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                         "value_one_core": len(ones) / sum(1.0 / v for v in ones),
                         "sample": "each step: " + res["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, power = [], [], []
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.file.read().splitlines():
            f = [x.strip() for x in row.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out.update({"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                        "samples": len(sm), "power_w_max": max(power)})
        return out


def measured_traffic(workload):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None if there
    is none for this workload or the kernel source has changed since the counters were taken."""
    import hashlib
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))[workload]
        src = open(os.path.join(ROOT, "paper_2502_13575_b200", "csrc", "ets_attn_narrow.cu"), "rb").read()
        if hashlib.sha256(src).hexdigest() != rec["kernel_source_sha256"]:
            return None
        return rec["dram_bytes_per_launch"]
    except Exception:
        return None


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- ranks
class RankComm:
    """The only inter-rank traffic of the benchmark: a barrier and a max-reduce of a scalar.
    Replicas are independent, so there is no data-path collective."""

    def __init__(self, world: int, device: str):
        self.world, self.device = world, device

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max_over_ranks(self, x: float) -> float:
        if self.world == 1:
            return x
        import torch
        import torch.distributed as dist
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def all_values(self, x: float):
        if self.world == 1:
            return [x]
        import torch
        import torch.distributed as dist
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        out = [torch.zeros_like(t) for _ in range(self.world)]
        dist.all_gather(out, t)
        return [float(o.item()) for o in out]


def replica_value_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own K/V/Q values; the tree is the same on every rank."""
    return base_seed + 7919 * rank


def aggregate_value(leaves_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job leaf-queries/s: what all ranks processed in a step over the slowest rank's time."""
    return world * leaves_per_rank / (ms_per_step / 1000.0)


# ----------------------------------------------------------------------------- probes and the per-workload table
TABLE_WORKLOADS = ("cfg1", "cfg2", "cfg3_diverse", "cfg3_ets", "cfg4", "cfg5a", "cfg5b", "cfg5c", "forest_w16x8", "forest_w64x8",
                   "search_w64_rebase", "search_w64_ets", "search_w256_rebase", "search_w256_ets")
NOMINAL_HBM_GBS = 8000.0


def _event_ms(torch, fn, reps):
    """Median over `reps` of the time of fn() between two events on the current stream."""
    out = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1))
    return statistics.median(out)


def run_probes(torch, device):
    """What the GPU gives a kernel of the streaming attention kernel's shape with no arithmetic (read-only, linear
    bulk copies into per-warp shared-memory rings), and what a launch costs."""
    import paper_2502_13575_b200 as ets
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    nbytes = 2 << 30                                  # far beyond L2: every launch reads from DRAM
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    buf.zero_()
    scratch = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    reads = []
    for chunk, depth in ((8192, 2), (8192, 3), (16384, 1), (4096, 4), (4096, 6), (2048, 8)):   # 8 warps x depth x chunk <= 227 KiB
        def launch():
            ets.ets_probe_stream_read(buf, nbytes, chunk, depth, sms, scratch, stream)
        for _ in range(3):
            launch()
        torch.cuda.synchronize()
        ms = _event_ms(torch, launch, 9)
        reads.append({"chunk_bytes": chunk, "copies_in_flight_per_warp": depth, "gbs": nbytes / (ms * 1e-3) / 1e9})
    if int(scratch[4096:4100].view(torch.int32).item()) != 0:
        raise RuntimeError("the streaming probe reported a wait that ran out")
    smem = 131200                                     # the streaming attention kernel's request at head_dim 128

    def one():
        ets.ets_probe_empty_launch(sms, smem, scratch, stream)
    for _ in range(20):
        one()
    torch.cuda.synchronize()
    single_us = _event_ms(torch, one, 51) * 1e3       # event, launch, event on an idle stream
    n = 200
    back_us = _event_ms(torch, lambda: [one() for _ in range(n)], 5) * 1e3 / n
    empty_us = _event_ms(torch, lambda: None, 51) * 1e3
    del buf
    return {
        "stream_read": reads,
        "stream_read_best_gbs": max(r["gbs"] for r in reads),
        "stream_read_attention_shape_gbs": reads[0]["gbs"],
        "what": f"{nbytes >> 20} MiB read once per launch by {sms} CTAs x 8 warps through linear bulk copies, no arithmetic",
        "launch": {"event_launch_event_us": single_us, "two_events_us": empty_us, "back_to_back_us_per_launch": back_us,
                   "what": f"empty kernel, {sms} CTAs x 256 threads, {smem} B dynamic shared memory"},
    }


def timeline_from_stamps(st, max_launches=64):
    """Mean timeline of a call from the library's device time stamps (ets_stamps_read), in microseconds relative to the
    start of the streaming attention kernel: when the append ahead of it ended, when its wait for that append returned,
    when it ended, the tcgen05 kernel's start and end (None without wide groups), the merge's end, and the period
    (merge end to merge end)."""
    cnt, s0, e0 = st["count"], st["start_ns"], st["end_ns"]
    n = int(min(cnt[1], cnt[3], cnt[4]))
    if n < 3:
        return None
    k = min(n - 1, max_launches)
    rows = []
    for j in range(n - k, n):
        def at(kind, arr):   # the launch of `kind` that belongs to the j-th launch counted from the end of the narrow series
            i = int(cnt[kind]) - (int(cnt[1]) - j)
            return None if i < 0 or i >= int(cnt[kind]) else int(arr[kind][i])
        base = at(1, s0)
        rec = {"append_start": at(0, s0), "append_end": at(0, e0), "narrow_wait_returned": at(4, s0), "narrow_end": at(1, e0),
               "wide_start": at(2, s0), "wide_end": at(2, e0), "merge_start": at(3, s0), "merge_end": at(3, e0)}
        rows.append({key: (None if v is None else (v - base) / 1e3) for key, v in rec.items()} | {"_merge_end_abs": at(3, e0)})
    out = {}
    for key in rows[0]:
        if key.startswith("_"):
            continue
        vals = [r[key] for r in rows if r[key] is not None]
        out[key] = float(np.mean(vals)) if len(vals) == len(rows) else None
    ends = [r["_merge_end_abs"] for r in rows]
    out["period"] = float(np.mean(np.diff(ends))) / 1e3
    out["launches"] = len(rows)
    return out


def measure_workload(torch, name, device, peak, probe_gbs, chain=None):
    """One row of the per-workload table: one tree, one layer per launch.  Cold protocol: the context holds R
    layers with R x (a layer's K/V) >= 4 x L2 and the launches rotate over them back to back, so a layer's K/V
    has left L2 when its turn comes again and launch latency hides behind the running kernels; for the two
    smallest trees R is capped and the note says so.  Beside it the time of a single call on an idle stream
    after L2 was overwritten."""
    import math
    import paper_2502_13575_b200 as ets
    from workloads import make_workload
    from workloads.loader import DecodeJob
    wl = make_workload(name)
    g, tree = wl.geometry, wl.tree
    L = tree.n_leaves
    U = int(tree.tokens.sum())
    l2 = torch.cuda.get_device_properties(device).L2_cache_size
    qo = 2 * L * g.num_q_heads * g.head_dim * 2
    layer_bytes = U * g.kv_bytes_per_token + qo
    R = int(min(32, max(2, math.ceil(4.0 * l2 / layer_bytes))))
    # iterations per timed loop: enough launches to time, few enough that the tree (one more token per leaf and
    # iteration) grows by a few percent only over the three loops
    n_tok, warm = int(max(4, min(math.ceil(192 / R), 0.01 * U / L))), 3
    job = DecodeJob(wl, headroom=4 * (n_tok + warm) + 16, device=device, layers=R, host_buffers=False, chain=chain)
    ctx = job.ctx
    # whole call (append + attention + merge) per layer: one decode iteration over the R layers captured into a
    # CUDA graph and replayed, so the host's launch rate is not what is measured
    replay = job.token_graph()
    replay(warm)
    torch.cuda.synchronize()

    def loop():
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        replay(n_tok)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    loops = []
    for _ in range(3):
        before = job.steps_done
        loops.append((loop() * 1e3 / (n_tok * R), U + L * (before + 0.5 * n_tok)))   # (us per call, mean unique tokens)
    call_us, u_call = min(loops)
    ctx.poll_status()
    # where a call's time goes: the same replayed loop with the kernels recording device time stamps
    ctx.set_option(ets.ETS_OPT_TIMING, 2)
    replay_stamped = job.token_graph()
    replay_stamped(warm)
    ctx.stamps_read()
    replay_stamped(n_tok)
    timeline = timeline_from_stamps(ctx.stamps_read(), max_launches=max(2, n_tok * R - 1))
    ctx.set_option(ets.ETS_OPT_TIMING, 0)
    del replay_stamped
    # the same calls launched one by one with events around the attention kernels and the merge kernel
    job.reset_lengths()
    ctx.set_option(ets.ETS_OPT_TIMING, 1)
    job.decode_tokens(warm)
    torch.cuda.synchronize()
    ctx.timing_read()
    job.decode_tokens(n_tok)
    torch.cuda.synchronize()
    attn_ms, merge_ms, n_calls = ctx.timing_read()
    ctx.set_option(ets.ETS_OPT_TIMING, 0)
    attn_us, merge_us = attn_ms * 1e3 / n_calls, merge_ms * 1e3 / n_calls
    # one call on an idle stream, L2 overwritten before it
    flush = torch.empty(2 * l2, dtype=torch.uint8, device="cuda")
    job.reset_lengths()
    p = job._pointers()
    stream = torch.cuda.current_stream().cuda_stream
    singles = []
    for i in range(9):
        flush.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.tree_attn_decode(i % R, p["q"][i % R], p["out"][i % R], None, stream=stream)
        e1.record()
        torch.cuda.synchronize()
        singles.append(e0.elapsed_time(e1) * 1e3)
    ctx.poll_status()
    # host time of a rebuild: a changed tree (the capacities alternate between two values, pages kept, so every call
    # flattens afresh and uploads), and the tree that is already current (recognised, nothing to do)
    cap_b = job.cap.copy()
    cap_b[tree.leaf_node] -= 1      # inside the pages the context was sized for; the tokens appended so far still fit
    t0 = time.perf_counter()
    for i in range(6):
        ctx.tree_build(tree.parent, cap_b if i % 2 == 0 else job.cap, tree.leaf_node, keep_pages_of=job.keep, stream=stream)
    flatten_ms = (time.perf_counter() - t0) / 6 * 1e3
    t0 = time.perf_counter()
    for _ in range(6):
        ctx.tree_build(tree.parent, job.cap, tree.leaf_node, keep_pages_of=job.keep, stream=stream)
    flatten_same_ms = (time.perf_counter() - t0) / 6 * 1e3
    torch.cuda.synchronize()
    st = ctx.get_stats()
    u_mean = U + L * (warm + 0.5 * (n_tok + 1))                          # every iteration appends one token per leaf
    alg = u_mean * g.kv_bytes_per_token + qo
    gbs = alg / (attn_us * 1e-6) / 1e9
    call_gbs = (u_call * g.kv_bytes_per_token + qo) / (call_us * 1e-6) / 1e9
    row = {
        "workload": name, "leaves": L, "unique_tokens": U, "algorithmic_bytes": alg,
        "layers_rotated": R, "cold": bool(R * layer_bytes >= 4 * l2),
        "attention_us": attn_us, "merge_us": merge_us, "gbs": gbs,
        "frac_measured_copy": gbs / peak, "frac_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
        "frac_read_probe": (gbs / probe_gbs) if probe_gbs else None,
        "call_us": call_us, "call_gbs": call_gbs, "call_frac_measured_copy": call_gbs / peak,
        "leaf_queries_per_s": L / (call_us * 1e-6),
        "single_call_after_flush_us": statistics.median(singles), "timeline_us": timeline,
        "flatten_host_ms": flatten_ms, "flatten_same_tree_host_ms": flatten_same_ms, "items": st["n_items"], "narrow_items": st["n_narrow_items"],
        "launches_timed": int(n_calls),
    }
    del job, flush
    torch.cuda.empty_cache()
    return row


def workload_table(torch, device, peak, probe_gbs, chain=None, names=TABLE_WORKLOADS):
    rows = [measure_workload(torch, n, device, peak, probe_gbs, chain) for n in names]
    by = {r["workload"]: r for r in rows}
    # the paper's claim on this kernel (Section 3, Table 2): a tree with 1.8x less KV should take about 1.8x less
    # time.  cfg3: the pair drawn with a keep fraction; search_*: the pairs grown by REBASE alone and by REBASE + the
    # library's ets_select, with the KV size of the whole search (sum over its steps) from the generator.
    from workloads import make_workload
    pair = {}
    for big, small, tag in (("cfg3_diverse", "cfg3_ets", "cfg3"), ("search_w64_rebase", "search_w64_ets", "search_w64"),
                            ("search_w256_rebase", "search_w256_ets", "search_w256")):
        if big not in by or small not in by:
            continue
        d, e = by[big], by[small]
        pair[tag + "_kv_ratio"] = d["unique_tokens"] / e["unique_tokens"]
        pair[tag + "_time_ratio_attention"] = d["attention_us"] / e["attention_us"]
        pair[tag + "_time_ratio_call"] = d["call_us"] / e["call_us"]
        if tag != "cfg3":
            pair[tag + "_search_kv_size_ratio"] = make_workload(small).notes["kv_ratio_vs_rebase"]
    note = ("one layer per launch; attention_us / merge_us: events around the attention kernels and the merge kernel in a "
            "back-to-back loop of ets_decode_step over layers_rotated layers (cold = those layers together exceed 4 x L2; the two "
            "smallest trees stay L2-resident); gbs and the frac_* columns divide algorithmic_bytes by attention_us; call_us: "
            "the whole call (append + attention + merge) per layer with the loop over the layers captured in a CUDA graph "
            "and replayed, no events inside, call_gbs from it; timeline_us: mean device time stamps of a call in the replayed "
            "loop, relative to the start of the streaming attention kernel (ETS_OPT_TIMING = 2); the cfg4 row is one layer "
            "of the headline workload in a context of layers_rotated layers")
    return {"rows": rows, "pair": pair, "note": note}


# ----------------------------------------------------------------------------- ours
def run_ours(args):
    import torch
    import torch.distributed as dist
    from workloads import make_workload
    from workloads.loader import DecodeJob
    import paper_2502_13575_b200 as ets

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    comm = RankComm(world, device="cuda")
    barrier, max_over_ranks = comm.barrier, comm.max_over_ranks

    wl = make_workload(args.workload)
    if rank:
        import dataclasses
        wl = dataclasses.replace(wl, value_seed=replica_value_seed(wl.value_seed, rank))
    g, tree = wl.geometry, wl.tree
    layers = args.layers or g.num_layers
    K, W = args.steps, args.warmup
    headroom = max(K + W + 2, args.loop_tokens + 4)
    job = DecodeJob(wl, headroom=headroom, device=local, layers=layers, chunk_pages=args.chunk_pages,
                    kernel=args.kernel, wide=args.wide, host_buffers=not args.no_e2e, chain=args.chain)
    ctx = job.ctx
    stats = ctx.get_stats()
    L = tree.n_leaves
    kv_bytes_tok = g.kv_bytes_per_token
    qo_bytes = 2 * L * g.num_q_heads * g.head_dim * 2

    # A step that streams less than a few L2 capacities would find its K/V still cached from the
    # previous step: then every step is timed on its own and L2 is overwritten in between.
    kv_bytes_step = float(tree.tokens.sum()) * kv_bytes_tok * layers
    l2_bytes = torch.cuda.get_device_properties(local).L2_cache_size
    flush = kv_bytes_step < 4 * l2_bytes
    flush_buf = torch.empty(max(2 * l2_bytes, 1 << 28), dtype=torch.uint8, device="cuda") if flush else None

    def timed_loop(step_fn, sync_each):
        job.reset_lengths()
        for _ in range(W):
            step_fn()
            if sync_each:
                torch.cuda.synchronize()
        u_tokens = []
        barrier()
        torch.cuda.synchronize()
        if not flush:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(K):
                step_fn()
                u_tokens.append(job.unique_tokens())
                if sync_each:
                    torch.cuda.synchronize()   # the host reads this step's result
            e1.record()
            torch.cuda.synchronize()
            ms_local = e0.elapsed_time(e1)
        else:
            pairs = []
            for _ in range(K):
                flush_buf.zero_()              # outside the timed region
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                step_fn()
                e1.record()
                u_tokens.append(job.unique_tokens())
                torch.cuda.synchronize()
                pairs.append((e0, e1))
            ms_local = sum(a.elapsed_time(b) for a, b in pairs)
        barrier()
        ms = max_over_ranks(ms_local)
        return ms, float(np.mean(u_tokens))

    # ---- device-resident throughput (the headline value) with clocks sampled during the region: the K-step
    # loop is timed `repeats` times, each one exactly K steps between a barrier + synchronise on both sides;
    # the reported step time is the median loop
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    loops = [timed_loop(job.step, sync_each=False) for _ in range(max(1, args.repeats))]
    clocks = sampler.stop() if rank == 0 else {}
    ctx.poll_status()
    loops.sort(key=lambda x: x[0])
    ms_total, u_mean = loops[len(loops) // 2]
    ms_step = ms_total / K
    value = aggregate_value(L, world, ms_step)
    repeats = {"loops": len(loops), "ms_per_step_median": ms_step, "ms_per_step_min": loops[0][0] / K,
               "ms_per_step_max": loops[-1][0] / K, "ms_per_step_all": [x[0] / K for x in loops]}

    # ---- same loop with the attention and merge kernels bracketed by events on their stream
    ctx.set_option(ets.ETS_OPT_TIMING, 1)
    job.reset_lengths()
    for _ in range(W):
        job.step()
    torch.cuda.synchronize()
    ctx.timing_read()
    u_tok2 = []
    for _ in range(K):
        if flush:
            flush_buf.zero_()
        job.step()
        u_tok2.append(job.unique_tokens())
    torch.cuda.synchronize()
    attn_ms, merge_ms, n_calls = ctx.timing_read()
    ctx.set_option(ets.ETS_OPT_TIMING, 0)
    attn_ms_per_launch = attn_ms / max(n_calls, 1)
    merge_ms_per_launch = merge_ms / max(n_calls, 1)
    alg_bytes_launch = float(np.mean(u_tok2)) * kv_bytes_tok + qo_bytes
    achieved = alg_bytes_launch / (attn_ms_per_launch * 1e-3) / 1e9
    peak, peak_kind = measured_hbm_peak()
    traffic = measured_traffic(args.workload)
    roofline = {
        "bound": "hbm", "kernel": "node-partial attention (narrow kernel, with the wide tcgen05 kernel overlapped)", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_kind": peak_kind + " copy bandwidth", "traffic": traffic,
        "algorithmic_bytes_per_launch": alg_bytes_launch, "us_per_launch": attn_ms_per_launch * 1e3,
        "merge_us_per_launch": merge_ms_per_launch * 1e3, "launches_timed": int(n_calls),
        "frac_of_nominal_8TBps": achieved / 8000.0,
        "whole_step_gbs": (u_mean * kv_bytes_tok + qo_bytes) * layers / (ms_step * 1e-3) / 1e9,
    }

    # ---- a search step's decode loop: one flatten, then T decode iterations of every layer through
    # ets_decode_step (append + attention in one call), no rebuild in between
    loop = None
    T = args.loop_tokens
    if T > 0:
        job.reset_lengths()
        job.decode_tokens(2)
        torch.cuda.synchronize()
        job.reset_lengths()
        barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.tree_build(tree.parent, job.cap, tree.leaf_node, keep_pages_of=job.keep,
                       stream=torch.cuda.current_stream().cuda_stream)
        job.decode_tokens(T)
        e1.record()
        torch.cuda.synchronize()
        ms_loop = max_over_ranks(e0.elapsed_time(e1))
        ctx.poll_status()
        loop = {"tokens": T, "ms_per_token": ms_loop / T, "leaf_tokens_per_s": world * L * T / (ms_loop / 1000.0),
                "what": "one ets_tree_build, then tokens x layers calls of ets_decode_step; device-resident inputs",
                "cache": "cold (a token streams more than L2 holds)" if not flush else
                         "warm: consecutive tokens find this tree's KV in L2"}

    # ---- end to end: host buffers through the *_host entry points, result read every step
    e2e = None
    if not args.no_e2e:
        ms_e2e, _ = timed_loop(job.step_host, sync_each=True)
        e2e = {"value": world * L / (ms_e2e / K / 1000.0), "unit": UNIT,
               "h2d_bytes_per_step": job.h2d_bytes_per_step, "d2h_bytes_per_step": job.d2h_bytes_per_step,
               "ms_per_step": ms_e2e / K}
    ctx.poll_status()

    # ---- the other workloads and the probes (default run only: one GPU, the headline workload)
    table = probes = None
    peak, peak_kind = measured_hbm_peak()
    if rank == 0 and world == 1 and not args.no_table and args.workload == "cfg4":
        del job
        torch.cuda.empty_cache()
        try:   # the headline line is printed whatever happens here
            probes = run_probes(torch, local)
            roofline["frac_of_read_probe"] = achieved / probes["stream_read_best_gbs"]
            table = workload_table(torch, local, peak, probes["stream_read_best_gbs"], chain=args.chain)
        except Exception as exc:   # noqa: BLE001
            table = {"error": f"{type(exc).__name__}: {exc}"}

    cpu = None
    if rank == 0 and not args.no_cpu_baseline and world == 1:
        res = oracle_sample(wl, layers, args.cpu_seconds)
        cpu = {"value": res["value"], "unit": UNIT, "cores": res["cores"], "kind": "oracle",
               "value_one_core": res["value_one_core"], "sample": res["sample"]}

    # kernels of the library per layer: append, narrow attention, merge, and the wide attention kernel when
    # the tree has wide query groups
    launches_per_layer = 3 + (1 if stats["n_items"] > stats["n_narrow_items"] else 0)
    if rank == 0:
        cfg = workload_description(wl, layers)
        cfg.update({"cache": ("L2 overwritten between steps (a step streams %.3f GB of KV); each step timed on its own"
                              if flush else "inputs larger than L2: every step streams %.2f GB of KV") %
                             (u_mean * kv_bytes_tok * layers / 1e9),
                    "parallelism": f"replicas x{world}, no collective",
                    "segments": stats["n_segments"], "chunks": stats["n_chunks"], "items": stats["n_items"]})
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": cfg, "clocks": clocks, "e2e": e2e,
            "gpu_launches": K * layers * launches_per_layer, "roofline": roofline, "cpu_baseline": cpu,
            "decode_loop": loop, "repeats": repeats, "workloads": table, "probes": probes,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_prefill(args):
    """Step-prefill attention on one GPU: every token of the last search step of the workload's tree is a
    query (a leaf on its step's node), one layer, K/V resident.  The work is a dense contraction (hundreds of
    query rows share every K/V tile), so the bound is the tensor pipe: 4 * d flops per (query row, visible token)."""
    import torch
    from workloads import make_workload, node_kv_bits, query_bits
    from paper_2502_13575_b200.runner import context_for_tree
    import paper_2502_13575_b200 as ets
    wl = make_workload(args.workload)
    tree, g = wl.tree, wl.geometry
    step_nodes = sorted(set(int(n) for n in tree.leaf_node))
    leaves = np.concatenate([np.full(int(tree.tokens[n]), n, np.int32) for n in step_nodes])
    limits = np.concatenate([np.arange(1, int(tree.tokens[n]) + 1, dtype=np.int32) for n in step_nodes])
    ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, tree.tokens, leaves)
    ctx.set_option(ets.ETS_OPT_WIDE, 17)
    ctx.set_option(ets.ETS_OPT_PATH_ITEMS, 0 if args.segment_items else 1)
    ctx.tree_build(tree.parent, tree.tokens, leaves)
    nodes = [n for n in range(tree.n_nodes) if tree.tokens[n] > 0]
    kv = [node_kv_bits(wl.value_seed, n, int(tree.tokens[n]), g.num_kv_heads, g.head_dim, 0) for n in nodes]
    k_all = torch.from_numpy(np.concatenate([x[0] for x in kv]).view(np.int16)).cuda().view(torch.bfloat16)
    v_all = torch.from_numpy(np.concatenate([x[1] for x in kv]).view(np.int16)).cuda().view(torch.bfloat16)
    ctx.kv_append(0, nodes, [int(tree.tokens[n]) for n in nodes], k_all, v_all)
    L = int(leaves.shape[0])
    q = torch.from_numpy(query_bits(wl.value_seed, 0, L, g.num_q_heads, g.head_dim).view(np.int16)).cuda().view(torch.bfloat16)
    out = torch.empty_like(q)
    lim = torch.from_numpy(limits).cuda()
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(args.warmup):
        ctx.tree_attn_prefill(0, q, lim, out, None, stream=stream)
    torch.cuda.synchronize()
    ctx.poll_status()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.tree_attn_prefill(0, q, lim, out, None, stream=stream)
    e1.record()
    torch.cuda.synchronize()
    ctx.poll_status()
    ms = e0.elapsed_time(e1) / args.steps
    # visible tokens per query: its ancestors' tokens plus its limit
    anc = np.zeros(tree.n_nodes, np.int64)
    for v in range(tree.n_nodes):
        p = int(tree.parent[v])
        anc[v] = (anc[p] + int(tree.tokens[p])) if p >= 0 else 0
    visible = int((anc[leaves] + limits).sum())
    flops = 4.0 * g.head_dim * visible * g.num_q_heads
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        peak, kind = float(peaks["bf16_tflops_sustained"]), "measured sustained cuBLAS bf16"
    except Exception:
        peak, kind = 1400.0, "fallback"
    st = ctx.get_stats()
    print(json.dumps({
        "metric": "step_prefill_attention_query_tokens_per_s", "value": L / (ms / 1000.0), "unit": "query-tokens/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload + " last step as queries", "query_tokens": L, "step_nodes": len(step_nodes),
                   "visible_tokens_per_query": visible / L, "heads": f"{g.num_q_heads}q/{g.num_kv_heads}kv x {g.head_dim}",
                   "layers": 1, "items": st["n_items"], "narrow_items_on_scalar_kernel": st["n_narrow_items"],
                   "decomposition": "segment items" if args.segment_items else "path items"},
        "roofline": {"bound": "tensor", "achieved": flops / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                     "frac": flops / (ms * 1e-3) / 1e12 / peak, "peak_kind": kind, "traffic": None,
                     "algorithmic_flops_per_launch": flops},
    }), flush=True)


def run_table_only(args):
    """Only the per-workload table and the probes, on one GPU."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    peak, peak_kind = measured_hbm_peak()
    names = tuple(n for n in args.table_workloads.split(",") if n) or TABLE_WORKLOADS
    probes = run_probes(torch, 0)
    table = workload_table(torch, 0, peak, probes["stream_read_best_gbs"], chain=args.chain, names=names)
    print(json.dumps({"workloads": table, "probes": probes, "peak": peak, "peak_kind": peak_kind + " copy bandwidth"}), flush=True)


def main():
    args = parse_args()
    if args.table_only:
        run_table_only(args)
    elif args.prefill:
        run_prefill(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
