"""Resident benchmark state: a context whose pools hold a seeded workload, plus the per-step
inputs of a decode step.  Shared by bench.py, the smoke check and the full-size GPU tests so
that all three drive the library in the same launch configuration.  It only moves data and
makes C-ABI calls; the attention arithmetic is in the library, the expected values in oracle/.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import numpy as np

from .trees import Workload
from .values import node_kv_bits, query_bits, layer_transform_bits


def base_rows(wl: Workload, lengths=None) -> Tuple[np.ndarray, np.ndarray, List[int], List[int]]:
    """Layer-0 K and V rows of every non-empty node, concatenated in node order."""
    tree, g = wl.tree, wl.geometry
    lengths = tree.tokens if lengths is None else lengths
    nodes = [n for n in range(tree.n_nodes) if int(lengths[n]) > 0]
    ks, vs = [], []
    for n in nodes:
        k, v = node_kv_bits(wl.value_seed, n, int(lengths[n]), g.num_kv_heads, g.head_dim, 0)
        ks.append(k)
        vs.append(v)
    return np.concatenate(ks), np.concatenate(vs), nodes, [int(lengths[n]) for n in nodes]


def layer_transform_torch(t_int16, layer: int):
    """The device-side twin of values.layer_transform_bits (rotate features, flip sign on odd layers)."""
    import torch
    if layer == 0:
        return t_int16
    out = torch.roll(t_int16, layer, dims=-1)
    if layer & 1:
        out = out ^ torch.tensor(-32768, dtype=torch.int16, device=out.device)
    return out


def step_token_bits(wl: Workload, layer: int, which: int) -> np.ndarray:
    """K (which=0) or V (which=1) rows of the token every leaf appends in a decode step:
    uint16 [n_leaves, num_kv_heads, head_dim].  The same rows are appended in every step."""
    g = wl.geometry
    k, v = node_kv_bits(wl.value_seed + 500000, 0, wl.tree.n_leaves, g.num_kv_heads, g.head_dim, 0)
    return layer_transform_bits(v if which else k, layer)


class DecodeJob:
    """One replica: pools filled with the workload, inputs of a decode step resident on the device
    (and mirrored in pinned host memory for the host-buffer entry points).

    A step is one pass of the whole path: tree flatten (all pages kept), then for every layer the
    append of one new token per leaf followed by tree-decode attention."""

    def __init__(self, wl: Workload, *, headroom: int, device: int = 0, layers: Optional[int] = None,
                 chunk_pages: Optional[int] = None, kernel: Optional[int] = None, wide: Optional[int] = None,
                 host_buffers: bool = True, chain: Optional[int] = None, overlap_append: int = 1):
        import torch
        from paper_2502_13575_b200.runner import context_for_tree
        import paper_2502_13575_b200 as ets
        self.torch, self.ets = torch, ets
        self.wl = wl
        tree, g = wl.tree, wl.geometry
        self.layers = g.num_layers if layers is None else layers
        self.dev = torch.device("cuda", device)
        self.cap = tree.tokens.copy()
        self.cap[tree.leaf_node] += headroom
        self.headroom = headroom
        self.steps_done = 0
        self.ctx = context_for_tree(g.num_q_heads, g.num_kv_heads, g.head_dim, tree.parent, self.cap,
                                    tree.leaf_node, num_layers=self.layers, device=device,
                                    chunk_pages=chunk_pages, extra_pages=8)
        if kernel is not None:
            self.ctx.set_option(ets.ETS_OPT_KERNEL, kernel)
        if wide is not None:
            self.ctx.set_option(ets.ETS_OPT_WIDE, wide)
        if chain is not None:
            self.ctx.set_option(ets.ETS_OPT_LAUNCH_CHAIN, chain)
        # the step inputs below are resident before any call: a call may start on them under the preceding merge kernel
        self.ctx.set_option(ets.ETS_OPT_OVERLAP_APPEND, overlap_append)
        self.ctx.set_option(ets.ETS_OPT_PACKED_INPUTS, 1)   # decode_tokens() packs k | v | q of a layer in one pinned buffer
        self.keep = np.arange(tree.n_nodes, dtype=np.int32)
        self.ctx.tree_build(tree.parent, self.cap, tree.leaf_node)
        # pools
        k0, v0, nodes, ntok = base_rows(wl)
        k0d = torch.from_numpy(k0.view(np.int16)).to(self.dev)
        v0d = torch.from_numpy(v0.view(np.int16)).to(self.dev)
        for layer in range(self.layers):
            kt = layer_transform_torch(k0d, layer).view(torch.bfloat16)
            vt = layer_transform_torch(v0d, layer).view(torch.bfloat16)
            self.ctx.kv_append(layer, nodes, ntok, kt, vt)
        torch.cuda.synchronize(self.dev)
        del k0d, v0d
        # per-step inputs
        L = tree.n_leaves
        qb = np.stack([query_bits(wl.value_seed, l, L, g.num_q_heads, g.head_dim) for l in range(self.layers)])
        nk = np.stack([step_token_bits(wl, l, 0) for l in range(self.layers)])
        nv = np.stack([step_token_bits(wl, l, 1) for l in range(self.layers)])
        self.q_bits, self.newk_bits, self.newv_bits = qb, nk, nv
        self.q = torch.from_numpy(qb.view(np.int16)).to(self.dev).view(torch.bfloat16)
        self.newk = torch.from_numpy(nk.view(np.int16)).to(self.dev).view(torch.bfloat16)
        self.newv = torch.from_numpy(nv.view(np.int16)).to(self.dev).view(torch.bfloat16)
        self.out = torch.empty_like(self.q)
        self.leaf_nodes = tree.leaf_node.astype(np.int32)
        self.ones = np.ones(L, np.int32)
        if host_buffers:
            self.ctx.set_option(ets.ETS_OPT_HOST_PIPELINE, 1)
            # per layer one pinned buffer [k_new | v_new | q], as a fused q/k/v projection would leave it
            kv_el = nk[0].size
            packed = torch.empty((self.layers, 2 * kv_el + qb[0].size), dtype=torch.int16).pin_memory()
            packed[:, :kv_el] = torch.from_numpy(nk.view(np.int16).reshape(self.layers, -1))
            packed[:, kv_el:2 * kv_el] = torch.from_numpy(nv.view(np.int16).reshape(self.layers, -1))
            packed[:, 2 * kv_el:] = torch.from_numpy(qb.view(np.int16).reshape(self.layers, -1))
            self.packed_h = packed
            self.newk_h = packed[:, :kv_el]
            self.newv_h = packed[:, kv_el:2 * kv_el]
            self.q_h = packed[:, 2 * kv_el:]
            self.out_h = torch.empty(qb.shape, dtype=torch.int16).pin_memory()
        torch.cuda.synchronize(self.dev)

    # bytes the caller moves per step through the host-buffer entry points
    @property
    def h2d_bytes_per_step(self) -> int:
        return int(self.q_bits.nbytes + self.newk_bits.nbytes + self.newv_bits.nbytes)

    @property
    def d2h_bytes_per_step(self) -> int:
        return int(self.q_bits.nbytes)

    def unique_tokens(self) -> int:
        return int(self.wl.tree.tokens.sum()) + self.wl.tree.n_leaves * self.steps_done

    def reset_lengths(self):
        """Clip every node back to the workload's own lengths (drops the appended step tokens)."""
        t = self.wl.tree
        self.ctx.tree_build(t.parent, t.tokens, t.leaf_node, keep_pages_of=self.keep)
        self.ctx.tree_build(t.parent, self.cap, t.leaf_node, keep_pages_of=self.keep)
        self.steps_done = 0

    def _pointers(self):
        """Raw addresses of the per-layer inputs and outputs, computed once: the step loop then costs
        two C calls per layer and no tensor slicing."""
        if getattr(self, "_ptrs", None) is None:
            L = self.layers
            p = {"q": [self.q[l].data_ptr() for l in range(L)], "out": [self.out[l].data_ptr() for l in range(L)],
                 "nk": [self.newk[l].data_ptr() for l in range(L)], "nv": [self.newv[l].data_ptr() for l in range(L)]}
            if hasattr(self, "q_h"):
                p.update({"q_h": [self.q_h[l].data_ptr() for l in range(L)],
                          "out_h": [self.out_h[l].data_ptr() for l in range(L)],
                          "nk_h": [self.newk_h[l].data_ptr() for l in range(L)],
                          "nv_h": [self.newv_h[l].data_ptr() for l in range(L)]})
            self._ptrs = p
        return self._ptrs

    def step(self):
        """Device-resident inputs: flatten + (append, attend) for every layer; all asynchronous."""
        if self.steps_done >= self.headroom:
            raise RuntimeError("step budget of this job exhausted; call reset_lengths()")
        t = self.wl.tree
        c = self.ctx
        p = self._pointers()
        stream = self.torch.cuda.current_stream().cuda_stream
        c.tree_build(t.parent, self.cap, t.leaf_node, keep_pages_of=self.keep, stream=stream)
        for layer in range(self.layers):
            c.decode_step(layer, p["nk"][layer], p["nv"][layer], p["q"][layer], p["out"][layer], None, stream=stream)
        self.steps_done += 1

    def decode_tokens(self, n_tokens: int):
        """A search step's decode loop: n_tokens iterations of (one new token per leaf, attention) over every
        layer through ets_decode_step, with no tree rebuild in between.  Asynchronous."""
        if self.steps_done + n_tokens > self.headroom:
            raise RuntimeError("step budget of this job exhausted; call reset_lengths()")
        c = self.ctx
        p = self._pointers()
        stream = self.torch.cuda.current_stream().cuda_stream
        for _ in range(n_tokens):
            for layer in range(self.layers):
                c.decode_step(layer, p["nk"][layer], p["nv"][layer], p["q"][layer], p["out"][layer], None, stream=stream)
        self.steps_done += n_tokens

    def token_graph(self):
        """One decode iteration over all layers (ets_decode_step per layer) captured into a CUDA graph.  Returns
        replay(n): n iterations with no host work per launch; the library's host-side lengths are kept in step
        with ets_note_decode_steps.  Needs two iterations of head room for the capture itself."""
        import gc
        torch = self.torch
        # one capture stream per job: the library orders its cached append list against the stream that uploaded it,
        # and a wait on that upload's event from another stream has no place inside a capture
        if getattr(self, "_graph_stream", None) is None:
            self._graph_stream = torch.cuda.Stream(device=self.dev)
        side = self._graph_stream
        with torch.cuda.stream(side):
            self.decode_tokens(1)      # an ordinary call first: it leaves the append's descriptor list on the device
        side.synchronize()
        gc.collect()                   # a context collected during the capture would synchronise the device inside it
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            self.decode_tokens(1)      # counted on the host, runs nothing: the first replay makes up for it
        state = {"owed": 1}

        def replay(n: int):
            if self.steps_done + n - state["owed"] > self.headroom:
                raise RuntimeError("step budget of this job exhausted")
            for _ in range(n):
                graph.replay()
            extra = n - state["owed"]
            state["owed"] = 0
            if extra > 0:
                for layer in range(self.layers):
                    self.ctx.note_decode_steps(layer, extra)
                self.steps_done += extra
        replay.graph = graph           # keeps the graph alive with the callable
        return replay

    def step_host(self):
        """Host buffers in, host buffers out: all layers of the step through one ets_decode_step_host_layers call
        (the layers' [k_new | v_new | q] records are one pinned buffer); the caller synchronises to read the result."""
        if self.steps_done >= self.headroom:
            raise RuntimeError("step budget of this job exhausted; call reset_lengths()")
        t = self.wl.tree
        c = self.ctx
        stream = self.torch.cuda.current_stream().cuda_stream
        c.tree_build(t.parent, self.cap, t.leaf_node, keep_pages_of=self.keep, stream=stream)
        c.decode_step_host_layers(0, self.layers, self.packed_h.data_ptr(), self.out_h.data_ptr(), None, stream=stream)
        c.host_join(stream=stream)   # the step's results are complete once this stream has passed here
        self.steps_done += 1

    def step_host_per_layer(self):
        """The same through one ets_decode_step_host call per layer."""
        if self.steps_done >= self.headroom:
            raise RuntimeError("step budget of this job exhausted; call reset_lengths()")
        t = self.wl.tree
        c = self.ctx
        p = self._pointers()
        stream = self.torch.cuda.current_stream().cuda_stream
        c.tree_build(t.parent, self.cap, t.leaf_node, keep_pages_of=self.keep, stream=stream)
        for layer in range(self.layers):
            c.decode_step_host(layer, p["nk_h"][layer], p["nv_h"][layer], p["q_h"][layer], p["out_h"][layer], None,
                               stream=stream)
        c.host_join(stream=stream)
        self.steps_done += 1

    # ---- what the oracle needs for a sample of leaves
    def oracle_inputs(self, layer: int, leaves):
        """(node_len, k_nodes, v_nodes) holding, for the nodes on the sampled leaves' paths, the
        rows the pools hold now: the workload's rows plus the tokens appended so far."""
        t, g = self.wl.tree, self.wl.geometry
        node_len = t.tokens.copy()
        node_len[t.leaf_node] += self.steps_done
        empty = np.zeros((0, g.num_kv_heads, g.head_dim), np.uint16)
        k_nodes = [empty] * t.n_nodes
        v_nodes = [empty] * t.n_nodes
        leaf_of_node = {int(n): i for i, n in enumerate(t.leaf_node)}
        for l in leaves:
            v = int(t.leaf_node[l])
            while v >= 0:
                if k_nodes[v] is empty and node_len[v] > 0:
                    k, vv = node_kv_bits(self.wl.value_seed, v, int(t.tokens[v]), g.num_kv_heads, g.head_dim, layer)
                    if v in leaf_of_node and self.steps_done:
                        i = leaf_of_node[v]
                        k = np.concatenate([k, np.repeat(self.newk_bits[layer, i][None], self.steps_done, 0)])
                        vv = np.concatenate([vv, np.repeat(self.newv_bits[layer, i][None], self.steps_done, 0)])
                    k_nodes[v], v_nodes[v] = k, vv
                v = int(t.parent[v])
        return node_len, k_nodes, v_nodes
