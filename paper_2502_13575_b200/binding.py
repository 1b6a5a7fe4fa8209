"""ctypes binding of the C ABI declared in include/ets.h.

Argument marshalling only: every step of the path (tree flatten, KV append, node-partial
attention, log-sum-exp merge) runs inside libets_b200.so.  Functions carry the C names.
PyTorch is used for device memory and streams, nothing else.  If the shared library is
missing this module raises at import time; there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

from . import build as _build

ETS_OK = 0
ETS_ERR_INVALID_ARG = -1
ETS_ERR_BAD_TREE = -2
ETS_ERR_POOL_EXHAUSTED = -3
ETS_ERR_UNSUPPORTED = -4
ETS_ERR_STATE = -5
ETS_ERR_CUDA = -6
ETS_ERR_DEVICE_TIMEOUT = -7

ETS_OPT_CHUNK_PAGES = 1
ETS_OPT_KERNEL = 2
ETS_OPT_TIMING = 3
ETS_OPT_WIDE = 4
ETS_OPT_HOST_PIPELINE = 6
ETS_OPT_PATH_ITEMS = 7
ETS_OPT_OVERLAP_APPEND = 8
ETS_OPT_PACKED_INPUTS = 9
ETS_OPT_LAUNCH_CHAIN = 10
ETS_OPT_TEST_FIRST_WAIT_POLLS = 11

_ERR_NAMES = {
    -1: "ETS_ERR_INVALID_ARG", -2: "ETS_ERR_BAD_TREE", -3: "ETS_ERR_POOL_EXHAUSTED",
    -4: "ETS_ERR_UNSUPPORTED", -5: "ETS_ERR_STATE", -6: "ETS_ERR_CUDA", -7: "ETS_ERR_DEVICE_TIMEOUT",
}


class EtsError(RuntimeError):
    def __init__(self, code: int, message: str = ""):
        self.code = int(code)
        super().__init__(f"{_ERR_NAMES.get(self.code, self.code)}: {message}")


class ets_config(C.Structure):
    _fields_ = [
        ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("page_size", C.c_int32), ("num_layers", C.c_int32), ("max_nodes", C.c_int32),
        ("max_leaves", C.c_int32), ("max_path_tokens", C.c_int32),
        ("max_path_entries", C.c_int64), ("pages_per_layer", C.c_int64),
        ("max_append_tokens", C.c_int32), ("device", C.c_int32), ("sm_scale", C.c_float),
        ("flags", C.c_int32),
    ]


_I32P = C.POINTER(C.c_int32)


class ets_tables_host(C.Structure):
    _fields_ = [
        ("n_nodes", C.c_int32), ("n_leaves", C.c_int32),
        ("n_pages", C.c_int64), ("n_group", C.c_int64), ("n_path", C.c_int64),
        ("node_page_off", _I32P), ("page_ids", _I32P), ("node_leaf_off", _I32P), ("node_leaves", _I32P),
        ("leaf_path_off", _I32P), ("leaf_path", _I32P), ("leaf_path_pos", _I32P),
        ("node_depth", _I32P), ("node_len", _I32P),
    ]


class ets_work_host(C.Structure):
    _fields_ = [
        ("n_units", C.c_int64), ("n_items", C.c_int64), ("n_leaf_slots", C.c_int64),
        ("n_partial_slots", C.c_int64), ("n_workers", C.c_int64),
        ("unit", _I32P), ("item", _I32P), ("leaf_slot_off", _I32P), ("leaf_slots", _I32P), ("worker_off", _I32P),
    ]


class ets_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "n_nodes", "n_leaves", "unique_tokens", "unique_kv_bytes", "path_tokens", "pages_used",
        "pages_free", "n_segments", "n_chunks", "n_items", "n_units", "n_partial_slots",
        "attended_tokens", "n_narrow_items")]


STAMP_KINDS, STAMP_LAUNCHES = 5, 4096


class ets_stamps_host(C.Structure):
    _fields_ = [("count", C.c_uint32 * 8), ("reserved", C.c_uint32 * 8),
                ("start_ns", C.c_uint64 * (STAMP_KINDS * STAMP_LAUNCHES)), ("end_ns", C.c_uint64 * (STAMP_KINDS * STAMP_LAUNCHES))]


class ets_select_params(C.Structure):
    _fields_ = [("temperature", C.c_double), ("lambda_b", C.c_double), ("lambda_d", C.c_double),
                ("width", C.c_int32), ("reserved", C.c_int32), ("node_limit", C.c_int64), ("node_tokens", _I32P)]


class ets_select_result(C.Structure):
    _fields_ = [("objective", C.c_double), ("nodes_explored", C.c_int64), ("proven_optimal", C.c_int32),
                ("n_kept", C.c_int32), ("n_nodes_kept", C.c_int32), ("reserved", C.c_int32),
                ("kv_tokens_kept", C.c_int64), ("kv_tokens_all", C.c_int64)]


# every symbol include/ets.h declares, with its C signature
_SIGNATURES = {
    "ets_pool_bytes": (C.c_int32, [C.POINTER(ets_config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "ets_create": (C.c_int32, [C.POINTER(ets_config), C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p)]),
    "ets_destroy": (C.c_int32, [C.c_void_p]),
    "ets_tree_build": (C.c_int32, [C.c_void_p, C.c_int32, _I32P, _I32P, _I32P, C.c_int32, _I32P, C.c_void_p]),
    "ets_tree_export": (C.c_int32, [C.c_void_p, C.POINTER(ets_tables_host)]),
    "ets_work_export": (C.c_int32, [C.c_void_p, C.POINTER(ets_work_host)]),
    "ets_kv_append": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, _I32P, _I32P, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_kv_append_host": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, _I32P, _I32P, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_get_node_len": (C.c_int32, [C.c_void_p, C.c_int32, _I32P]),
    "ets_tree_attn_decode": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_select": (C.c_int32, [C.c_int32, _I32P, C.c_int32, _I32P, C.POINTER(C.c_double), _I32P,
                               C.POINTER(ets_select_params), _I32P, _I32P, _I32P, _I32P, C.POINTER(ets_select_result)]),
    "ets_tree_attn_prefill": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p]),
    "ets_decode_step": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p]),
    "ets_note_decode_steps": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32]),
    "ets_decode_step_host": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p]),
    "ets_decode_step_host_layers": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_tree_attn_decode_host": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_tree_attn_decode_static": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_kv_read_debug": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ets_get_stats": (C.c_int32, [C.c_void_p, C.POINTER(ets_stats)]),
    "ets_set_option": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int64]),
    "ets_host_join": (C.c_int32, [C.c_void_p, C.c_void_p]),
    "ets_timing_read": (C.c_int32, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "ets_stamps_read": (C.c_int32, [C.c_void_p, C.POINTER(ets_stamps_host)]),
    "ets_poll_status": (C.c_int32, [C.c_void_p, C.c_void_p]),
    "ets_probe_stream_read": (C.c_int32, [C.c_void_p, C.c_size_t, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "ets_probe_empty_launch": (C.c_int32, [C.c_int32, C.c_size_t, C.c_void_p, C.c_void_p]),
    "ets_last_error": (C.c_char_p, [C.c_void_p]),
    "ets_version": (C.c_char_p, []),
}


def _load() -> C.CDLL:
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2502_13575_b200.build` "
            "(there is no fallback path)")
    lib = C.CDLL(path)
    for name, (res, args) in _SIGNATURES.items():
        fn = getattr(lib, name)  # AttributeError if the library does not export it
        fn.restype = res
        fn.argtypes = args
    return lib


lib = _load()


def _i32(a) -> np.ndarray:
    if isinstance(a, np.ndarray) and a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]:
        return a
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: Optional[np.ndarray]):
    # a raw address converts faster than numpy's ctypes view and is accepted for POINTER arguments
    return None if a is None else C.cast(a.__array_interface__["data"][0], _I32P)


def _dev_ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array / raw int; None passes NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        if torch.cuda.is_available():
            return torch.cuda.current_stream().cuda_stream or None
        return None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def make_config(num_q_heads: int, num_kv_heads: int, head_dim: int, *, num_layers: int = 1,
                max_nodes: int, max_leaves: int, max_path_tokens: int, max_path_entries: int,
                pages_per_layer: int, page_size: int = 16, max_append_tokens: int = 0,
                device: int = 0, sm_scale: float = 0.0) -> ets_config:
    return ets_config(num_q_heads, num_kv_heads, head_dim, page_size, num_layers, max_nodes, max_leaves,
                      max_path_tokens, max_path_entries, pages_per_layer, max_append_tokens, device,
                      sm_scale, 0)


def ets_version() -> str:
    return lib.ets_version().decode()


def ets_select(parent, leaf_node, reward, cluster=None, *, width: int, temperature: float = 0.2,
               lambda_b: float = 0.0, lambda_d: float = 0.0, node_limit: int = 0, node_tokens=None) -> Dict[str, object]:
    """Selection step on the host (same name as the C call): REBASE weights, the kept set, the
    continuations per kept trajectory and the kept nodes of the tree."""
    parent, leaves = _i32(parent), _i32(leaf_node)
    r = np.ascontiguousarray(reward, dtype=np.float64)
    cl = None if cluster is None else _i32(cluster)
    tok = None if node_tokens is None else _i32(node_tokens)
    prm = ets_select_params(temperature, lambda_b, lambda_d, width, 0, node_limit, _p(tok))
    res = ets_select_result()
    L, n = leaves.shape[0], parent.shape[0]
    weight, keep, cont, nodes = (np.zeros(L, np.int32), np.zeros(L, np.int32), np.zeros(L, np.int32),
                                 np.zeros(n, np.int32))
    rc = lib.ets_select(n, _p(parent), L, _p(leaves), r.ctypes.data_as(C.POINTER(C.c_double)), _p(cl), C.byref(prm),
                        _p(weight), _p(keep), _p(cont), _p(nodes), C.byref(res))
    if rc != ETS_OK:
        raise EtsError(rc, "ets_select")
    return {"weight": weight, "keep": keep, "continuations": cont, "node_kept": nodes, "objective": res.objective,
            "proven_optimal": bool(res.proven_optimal), "nodes_explored": int(res.nodes_explored),
            "n_kept": int(res.n_kept), "n_nodes_kept": int(res.n_nodes_kept),
            "kv_tokens_kept": int(res.kv_tokens_kept), "kv_tokens_all": int(res.kv_tokens_all)}


def ets_probe_stream_read(buf, nbytes: int, chunk_bytes: int, depth: int, n_ctas: int, scratch, stream=None):
    """Measurement probe (same name as the C call): streams `nbytes` of `buf` once through the bulk-copy ring."""
    rc = lib.ets_probe_stream_read(_dev_ptr(buf), nbytes, chunk_bytes, depth, n_ctas, _dev_ptr(scratch), _stream_ptr(stream))
    if rc != ETS_OK:
        raise EtsError(rc, "ets_probe_stream_read")


def ets_probe_empty_launch(n_ctas: int, smem_bytes: int, scratch, stream=None):
    """Measurement probe (same name as the C call): launches a kernel that does nothing."""
    rc = lib.ets_probe_empty_launch(n_ctas, smem_bytes, _dev_ptr(scratch), _stream_ptr(stream))
    if rc != ETS_OK:
        raise EtsError(rc, "ets_probe_empty_launch")


def ets_pool_bytes(cfg: ets_config):
    k, v, w = C.c_size_t(), C.c_size_t(), C.c_size_t()
    rc = lib.ets_pool_bytes(C.byref(cfg), C.byref(k), C.byref(v), C.byref(w))
    if rc != ETS_OK:
        raise EtsError(rc, "ets_pool_bytes")
    return k.value, v.value, w.value


class EtsContext:
    """Owns the device buffers (torch allocations) and the opaque ets_ctx handle.  Method names
    are the C entry points without the `ets_` prefix; each one is a single C call."""

    def __init__(self, cfg: ets_config):
        self.cfg = cfg
        self._h = C.c_void_p()
        kb, vb, wb = ets_pool_bytes(cfg)
        self.k_pool = self.v_pool = self.workspace = None
        if cfg.device >= 0:
            import torch
            dev = torch.device("cuda", cfg.device)
            def aligned(nbytes):   # torch hands out small blocks on 512-byte boundaries; the library wants 1024
                t = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
                off = (-t.data_ptr()) % 1024
                return t[off:off + nbytes]
            self.k_pool, self.v_pool, self.workspace = aligned(kb), aligned(vb), aligned(wb)
        rc = lib.ets_create(C.byref(cfg), _dev_ptr(self.k_pool), _dev_ptr(self.v_pool),
                            _dev_ptr(self.workspace), C.byref(self._h))
        if rc != ETS_OK:
            raise EtsError(rc, "ets_create")

    # -- plumbing
    def _check(self, rc: int):
        if rc != ETS_OK:
            raise EtsError(rc, lib.ets_last_error(self._h).decode())

    def close(self):
        if self._h:
            lib.ets_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C entry points
    def tree_build(self, parent, cap_tokens, leaf_node, keep_pages_of=None, stream=None):
        parent, cap, leaves = _i32(parent), _i32(cap_tokens), _i32(leaf_node)
        keep = None if keep_pages_of is None else _i32(keep_pages_of)
        if cap.shape != parent.shape or (keep is not None and keep.shape != parent.shape):
            raise EtsError(ETS_ERR_INVALID_ARG, "array lengths differ")
        self._check(lib.ets_tree_build(self._h, parent.shape[0], _p(parent), _p(cap), _p(keep),
                                       leaves.shape[0], _p(leaves), _stream_ptr(stream)))

    def tree_export(self) -> Dict[str, np.ndarray]:
        t = ets_tables_host()
        self._check(lib.ets_tree_export(self._h, C.byref(t)))
        sizes = {
            "node_page_off": t.n_nodes + 1, "page_ids": t.n_pages, "node_leaf_off": t.n_nodes + 1,
            "node_leaves": t.n_group, "leaf_path_off": t.n_leaves + 1, "leaf_path": t.n_path,
            "leaf_path_pos": t.n_path, "node_depth": t.n_nodes, "node_len": t.n_nodes,
        }
        out = {k: np.zeros(n, dtype=np.int32) for k, n in sizes.items()}
        for k, a in out.items():
            setattr(t, k, _p(a))
        self._check(lib.ets_tree_export(self._h, C.byref(t)))
        return out

    def work_export(self) -> Dict[str, np.ndarray]:
        w = ets_work_host()
        self._check(lib.ets_work_export(self._h, C.byref(w)))
        n_lists = self.get_stats()["n_leaves"] * self.cfg.num_kv_heads
        out = {
            "unit": np.zeros(w.n_units * 4, np.int32), "item": np.zeros(w.n_items * 8, np.int32),
            "leaf_slot_off": np.zeros(n_lists + 1, np.int32), "leaf_slots": np.zeros(w.n_leaf_slots, np.int32),
            "worker_off": np.zeros(w.n_workers + 1, np.int32),
        }
        for k, a in out.items():
            setattr(w, k, _p(a))
        self._check(lib.ets_work_export(self._h, C.byref(w)))
        out["unit"] = out["unit"].reshape(-1, 4)
        out["item"] = out["item"].reshape(-1, 8)
        out["n_partial_slots"] = int(w.n_partial_slots)
        return out

    def get_node_len(self, layer: int = 0) -> np.ndarray:
        n = self.get_stats()["n_nodes"]
        a = np.zeros(n, np.int32)
        self._check(lib.ets_get_node_len(self._h, layer, _p(a)))
        return a

    def kv_append(self, layer: int, node_id, n_new, k_new, v_new, stream=None):
        node_id, n_new = _i32(node_id), _i32(n_new)
        self._check(lib.ets_kv_append(self._h, layer, node_id.shape[0], _p(node_id), _p(n_new),
                                      _dev_ptr(k_new), _dev_ptr(v_new), _stream_ptr(stream)))

    def kv_append_host(self, layer: int, node_id, n_new, k_new, v_new, stream=None):
        node_id, n_new = _i32(node_id), _i32(n_new)
        self._check(lib.ets_kv_append_host(self._h, layer, node_id.shape[0], _p(node_id), _p(n_new),
                                           _dev_ptr(k_new), _dev_ptr(v_new), _stream_ptr(stream)))

    def tree_attn_decode(self, layer: int, q, out, lse=None, stream=None):
        self._check(lib.ets_tree_attn_decode(self._h, layer, _dev_ptr(q), _dev_ptr(out), _dev_ptr(lse),
                                             _stream_ptr(stream)))

    def tree_attn_prefill(self, layer: int, q, leaf_limit, out, lse=None, stream=None):
        self._check(lib.ets_tree_attn_prefill(self._h, layer, _dev_ptr(q), _dev_ptr(leaf_limit), _dev_ptr(out),
                                              _dev_ptr(lse), _stream_ptr(stream)))

    def decode_step(self, layer: int, k_new, v_new, q, out, lse=None, stream=None):
        self._check(lib.ets_decode_step(self._h, layer, _dev_ptr(k_new), _dev_ptr(v_new), _dev_ptr(q), _dev_ptr(out),
                                        _dev_ptr(lse), _stream_ptr(stream)))

    def note_decode_steps(self, layer: int, times: int):
        self._check(lib.ets_note_decode_steps(self._h, layer, times))

    def decode_step_host(self, layer: int, k_new, v_new, q, out, lse=None, stream=None):
        self._check(lib.ets_decode_step_host(self._h, layer, _dev_ptr(k_new), _dev_ptr(v_new), _dev_ptr(q),
                                             _dev_ptr(out), _dev_ptr(lse), _stream_ptr(stream)))

    def decode_step_host_layers(self, first_layer: int, n_layers: int, inputs, out, lse=None, stream=None):
        self._check(lib.ets_decode_step_host_layers(self._h, first_layer, n_layers, _dev_ptr(inputs), _dev_ptr(out),
                                                    _dev_ptr(lse), _stream_ptr(stream)))

    def tree_attn_decode_host(self, layer: int, q, out, lse=None, stream=None):
        self._check(lib.ets_tree_attn_decode_host(self._h, layer, _dev_ptr(q), _dev_ptr(out), _dev_ptr(lse),
                                                  _stream_ptr(stream)))

    def tree_attn_decode_static(self, layer: int, q, out, lse=None, stream=None):
        """Decode using the library's built-in 8 MiB scratch: for callers that may not allocate
        device memory.  Small trees only; calls on one GPU must not overlap."""
        self._check(lib.ets_tree_attn_decode_static(self._h, layer, _dev_ptr(q), _dev_ptr(out), _dev_ptr(lse),
                                                    _stream_ptr(stream)))

    def kv_read_debug(self, layer: int, node: int, k_out, v_out, stream=None):
        self._check(lib.ets_kv_read_debug(self._h, layer, node, _dev_ptr(k_out), _dev_ptr(v_out),
                                          _stream_ptr(stream)))

    def get_stats(self) -> Dict[str, int]:
        s = ets_stats()
        self._check(lib.ets_get_stats(self._h, C.byref(s)))
        return {n: int(getattr(s, n)) for n, _ in ets_stats._fields_}

    def set_option(self, key: int, value: int):
        self._check(lib.ets_set_option(self._h, key, value))

    def host_join(self, stream=None):
        self._check(lib.ets_host_join(self._h, _stream_ptr(stream)))

    def timing_read(self):
        a, m, n = C.c_double(), C.c_double(), C.c_int64()
        self._check(lib.ets_timing_read(self._h, C.byref(a), C.byref(m), C.byref(n)))
        return a.value, m.value, n.value

    def stamps_read(self) -> Dict[str, np.ndarray]:
        """Device time stamps since the last read: counts [5] and, per kind, start / end in ns ([5, launches])."""
        st = ets_stamps_host()
        self._check(lib.ets_stamps_read(self._h, C.byref(st)))
        count = np.array(list(st.count)[:STAMP_KINDS], dtype=np.int64)
        start = np.ctypeslib.as_array(st.start_ns).reshape(STAMP_KINDS, STAMP_LAUNCHES).astype(np.int64)
        end = np.ctypeslib.as_array(st.end_ns).reshape(STAMP_KINDS, STAMP_LAUNCHES).astype(np.int64)
        return {"count": count, "start_ns": start.copy(), "end_ns": end.copy()}

    def poll_status(self, stream=None):
        self._check(lib.ets_poll_status(self._h, _stream_ptr(stream)))
