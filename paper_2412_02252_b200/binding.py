"""Thin ctypes binding of the C ABI declared in ``include/pod.h``.

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
Tensors are passed as raw device pointers (``tensor.data_ptr()``); PyTorch supplies device
memory and streams, nothing else.  There is no fallback: if the shared library is missing
and cannot be built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

from . import build as _build

POD_OK, POD_DRY_RUN = 0, 1
POD_ERR_INVALID, POD_ERR_CAPACITY, POD_ERR_ORDER = -1, -2, -3
POD_ERR_ARENA, POD_ERR_CUDA, POD_ERR_DEVICE = -4, -5, -6
POD_BYTES_LIVE, POD_BYTES_DENSE_EQUIV, POD_BYTES_ALLOCATED = 0, 1, 2
(POD_REGION_SINK_K, POD_REGION_SINK_V, POD_REGION_RING_K, POD_REGION_RING_V,
 POD_REGION_DIST_K, POD_REGION_DIST_V) = range(6)


class pod_config(ctypes.Structure):
    _fields_ = [("n_layers", c_int32), ("n_q_heads", c_int32), ("n_kv_heads", c_int32),
                ("head_dim", c_int32), ("group_size", c_int32), ("n_sink", c_int32),
                ("n_recent", c_int32), ("batch", c_int32), ("sm_scale", c_float),
                ("device", c_int32)]


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path) or _build.needs_build():
        try:
            path = _build.build()
        except Exception as e:  # no nvcc where the library is missing: fail loudly
            if not os.path.exists(path):
                raise ImportError(f"libpod_b200.so is missing and could not be built: {e}") from e
    lib = ctypes.CDLL(path)
    P = POINTER
    sig = {
        "pod_cache_required_bytes": (c_size_t, [P(pod_config), P(c_int32)]),
        "pod_cache_create": (c_int, [P(pod_config), P(c_int32), c_void_p, c_size_t, P(c_void_p)]),
        "pod_cache_required_bytes_blocks": (c_size_t, [P(pod_config), P(c_int32), P(c_int32)]),
        "pod_cache_create_blocks": (c_int, [P(pod_config), P(c_int32), P(c_int32), c_void_p, c_size_t, P(c_void_p)]),
        "pod_greedy_layer_blocks": (c_int, [P(c_float), c_int, c_int, c_float, P(c_int32)]),
        "pod_shard_config": (c_int, [P(pod_config), c_int, c_int, P(pod_config), P(c_int32), P(c_int32)]),
        "pod_shard_block_map": (c_int, [P(pod_config), P(c_int32), c_int, c_int, P(c_int32)]),
        "pod_cache_destroy": (c_int, [c_void_p]),
        "pod_cache_write": (c_int, [c_void_p, c_int, c_int, c_void_p, c_void_p, c_int, c_void_p]),
        "pod_decode_attn": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_void_p]),
        "pod_append_decode_attn": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
        "pod_cache_set_gate_threshold": (c_int, [c_void_p, c_float]),
        "pod_cache_bytes": (c_int64, [c_void_p, c_int]),
        "pod_cache_seq_len": (c_int, [c_void_p, c_int, c_int]),
        "pod_cache_reset": (c_int, [c_void_p, c_int]),
        "pod_cache_read_region": (c_int, [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int, c_void_p]),
        "pod_cache_device_status": (c_int, [c_void_p]),
        "pod_cache_inject_error": (c_int, [c_void_p]),
        "pod_cache_inject_stale_query": (c_int, [c_void_p]),
        "pod_cache_last_cuda_error": (c_int, [c_void_p]),
        "pod_cache_last_launch": (c_int, [c_void_p, P(c_int32), P(c_int32), P(c_int32)]),
        "pod_cache_set_trace": (c_int, [c_void_p, c_void_p, c_int]),
        "pod_cache_trace_count": (c_int, [c_void_p]),
        "pod_strerror": (c_char_p, [c_int]),
        "pod_prefill_attn": (c_int, [c_int, c_int, c_int, c_int, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p,
                                     c_void_p, c_void_p, P(c_int32), c_void_p, c_void_p]),
        "pod_prefill_status": (c_int, []),
        "pod_prefill_inject_error": (c_int, []),
        "pod_dense_decode_attn_static": (c_int, [c_void_p, c_int, c_int, c_void_p, c_void_p, c_int, c_int,
                                                 c_int, c_float, c_void_p]),
        "pod_dense_decode_attn_static_status": (c_int, []),
        "pod_dense_decode_attn_static_inject_error": (c_int, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()
EXPORTS = ["pod_cache_required_bytes", "pod_cache_create", "pod_cache_required_bytes_blocks",
           "pod_cache_create_blocks", "pod_greedy_layer_blocks", "pod_shard_config", "pod_shard_block_map",
           "pod_cache_destroy", "pod_cache_write",
           "pod_decode_attn", "pod_append_decode_attn", "pod_cache_set_gate_threshold", "pod_cache_bytes", "pod_cache_seq_len", "pod_cache_reset",
           "pod_cache_read_region", "pod_cache_device_status", "pod_cache_inject_error", "pod_cache_inject_stale_query",
           "pod_cache_last_cuda_error",
           "pod_cache_last_launch", "pod_cache_set_trace", "pod_cache_trace_count", "pod_strerror", "pod_prefill_attn", "pod_prefill_status", "pod_prefill_inject_error",
           "pod_dense_decode_attn_static", "pod_dense_decode_attn_static_status",
           "pod_dense_decode_attn_static_inject_error"]


class PodError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {pod_strerror(status)} ({status})")


def pod_strerror(status: int) -> str:
    return lib.pod_strerror(status).decode()


def _check(status: int, where: str) -> int:
    if status < 0:
        raise PodError(status, where)
    return status


def _ptr(t) -> int:
    return 0 if t is None else (t if isinstance(t, int) else t.data_ptr())


def make_config(*, n_layers, n_q_heads, n_kv_heads, head_dim, group_size, n_sink, n_recent, batch,
                sm_scale=0.0, device=0) -> pod_config:
    return pod_config(n_layers, n_q_heads, n_kv_heads, head_dim, group_size, n_sink, n_recent,
                      batch, sm_scale, device)


def _caps(cfg: pod_config, seq_capacity):
    caps = list(seq_capacity)
    if len(caps) != cfg.batch:
        raise ValueError("one capacity per sequence")
    return (c_int32 * cfg.batch)(*caps)


def _lowest(cfg: pod_config, lowest_layer):
    """[n_layers][n_kv_heads] nested sequence (or array) -> flat c_int32 array."""
    flat = [int(x) for row in lowest_layer for x in row]
    if len(flat) != cfg.n_layers * cfg.n_kv_heads:
        raise ValueError("lowest_layer must be [n_layers][n_kv_heads]")
    return (c_int32 * len(flat))(*flat)


def pod_cache_required_bytes(cfg: pod_config, seq_capacity, lowest_layer=None) -> int:
    if lowest_layer is None:
        return lib.pod_cache_required_bytes(ctypes.byref(cfg), _caps(cfg, seq_capacity))
    return lib.pod_cache_required_bytes_blocks(ctypes.byref(cfg), _caps(cfg, seq_capacity), _lowest(cfg, lowest_layer))


def pod_greedy_layer_blocks(sim, threshold: float = 0.5):
    """sim: nested sequence / array [n_heads][n_layers][n_layers]; returns lowest_layer as a list
    [n_layers][n_heads] of ints."""
    H, L = len(sim), len(sim[0])
    flat = (c_float * (H * L * L))(*[float(x) for a in sim for row in a for x in row])
    out = (c_int32 * (L * H))()
    _check(lib.pod_greedy_layer_blocks(flat, H, L, threshold, out), "pod_greedy_layer_blocks")
    return [[out[l * H + h] for h in range(H)] for l in range(L)]


def pod_shard_config(cfg: pod_config, rank: int, world: int):
    """KV-head split: returns (local config, first KV head, first query head) of ``rank``."""
    local, kv0, q0 = pod_config(), c_int32(), c_int32()
    _check(lib.pod_shard_config(ctypes.byref(cfg), rank, world, ctypes.byref(local), ctypes.byref(kv0), ctypes.byref(q0)),
           "pod_shard_config")
    return local, kv0.value, q0.value


def pod_shard_block_map(cfg: pod_config, lowest_layer, rank: int, world: int):
    """The rank's columns of a head-wise block map, as a list [n_layers][n_kv_heads / world]."""
    per = cfg.n_kv_heads // max(world, 1)
    out = (c_int32 * max(1, cfg.n_layers * per))()
    _check(lib.pod_shard_block_map(ctypes.byref(cfg), _lowest(cfg, lowest_layer), rank, world, out), "pod_shard_block_map")
    return [[out[l * per + h] for h in range(per)] for l in range(cfg.n_layers)]


class PodCache:
    """Owner of one ``pod_cache*``; methods carry the C names without the prefix."""

    def __init__(self, cfg: pod_config, seq_capacity, arena=None, lowest_layer=None):
        self.cfg = cfg
        self._arena = arena                       # keeps the caller's tensor alive
        handle = c_void_p()
        nbytes = 0 if arena is None else arena.numel() * arena.element_size()
        if lowest_layer is None:
            st = lib.pod_cache_create(ctypes.byref(cfg), _caps(cfg, seq_capacity), _ptr(arena), nbytes,
                                      ctypes.byref(handle))
            _check(st, "pod_cache_create")
        else:
            st = lib.pod_cache_create_blocks(ctypes.byref(cfg), _caps(cfg, seq_capacity), _lowest(cfg, lowest_layer),
                                             _ptr(arena), nbytes, ctypes.byref(handle))
            _check(st, "pod_cache_create_blocks")
        self._h = handle

    def destroy(self):
        if self._h is not None:
            h, self._h = self._h, None
            _check(lib.pod_cache_destroy(h), "pod_cache_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def write(self, layer: int, seq: int, k, v, n_tokens: int, stream: int = 0) -> int:
        return _check(lib.pod_cache_write(self._h, layer, seq, _ptr(k), _ptr(v), n_tokens, stream),
                      "pod_cache_write")

    def decode_attn(self, layer: int, q, out, stream: int = 0) -> int:
        return _check(lib.pod_decode_attn(self._h, layer, _ptr(q), _ptr(out), stream), "pod_decode_attn")

    def append_decode_attn(self, layer: int, k, v, q, out, stream: int = 0) -> int:
        return _check(lib.pod_append_decode_attn(self._h, layer, _ptr(k), _ptr(v), _ptr(q), _ptr(out), stream),
                      "pod_append_decode_attn")

    def set_gate_threshold(self, tau: float) -> int:
        return _check(lib.pod_cache_set_gate_threshold(self._h, tau), "pod_cache_set_gate_threshold")

    def bytes(self, which: int) -> int:
        return lib.pod_cache_bytes(self._h, which)

    def seq_len(self, seq: int, layer: int) -> int:
        return _check(lib.pod_cache_seq_len(self._h, seq, layer), "pod_cache_seq_len")

    def reset(self, seq: int = -1) -> int:
        return _check(lib.pod_cache_reset(self._h, seq), "pod_cache_reset")

    def read_region(self, region: int, layer_or_block: int, seq: int, kv_head: int, first: int, count: int):
        """Returns a numpy uint16 array [count][head_dim] of bf16 bit patterns."""
        import numpy as np
        dst = np.empty((count, self.cfg.head_dim), dtype=np.uint16)
        _check(lib.pod_cache_read_region(self._h, region, layer_or_block, seq, kv_head, first, count,
                                         dst.ctypes.data), "pod_cache_read_region")
        return dst

    def device_status(self) -> int:
        return lib.pod_cache_device_status(self._h)

    def inject_error(self) -> int:
        """Sets the cache's error word from the host (tests of the error path)."""
        return _check(lib.pod_cache_inject_error(self._h), "pod_cache_inject_error")

    def inject_stale_query(self) -> int:
        """The next decode launch recomputes every head as if its early copy of q had been stale (test hook)."""
        return _check(lib.pod_cache_inject_stale_query(self._h), "pod_cache_inject_stale_query")

    def last_cuda_error(self) -> int:
        return lib.pod_cache_last_cuda_error(self._h)

    def set_trace(self, pairs, n_launches: int) -> int:
        """pairs: int64/uint64 device tensor of 2 * n_launches elements (or None, 0 to switch off)."""
        return _check(lib.pod_cache_set_trace(self._h, _ptr(pairs), n_launches), "pod_cache_set_trace")

    def trace_count(self) -> int:
        return lib.pod_cache_trace_count(self._h)

    def last_launch(self):
        a, b, c = c_int32(), c_int32(), c_int32()
        lib.pod_cache_last_launch(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
        return {"split_tokens": a.value, "n_ctas": b.value, "n_kernels": c.value}


def pod_prefill_attn(q, k, v, out, *, n_sink: int, n_recent: int, q_low=None, k_low=None, head_shares=None,
                     sm_scale: float = 0.0, stream: int = 0) -> int:
    """PoD attention for every position (prefill) from dense bf16 projections ``q`` [T][H_q][d] (d 64 or 128),
    ``k``, ``v`` [T][H_kv][d]; ``q_low``/``k_low``: the lowest layer's, for layers that share."""
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    hs = None if head_shares is None else (c_int32 * Hkv)(*[int(x) for x in head_shares])
    return _check(lib.pod_prefill_attn(T, Hq, Hkv, d, n_sink, n_recent, sm_scale, _ptr(q), _ptr(k), _ptr(v),
                                       _ptr(q_low), _ptr(k_low), hs, _ptr(out), stream), "pod_prefill_attn")


def pod_prefill_status() -> int:
    return lib.pod_prefill_status()


def pod_prefill_inject_error() -> int:
    """Sets the device's prefill error word from the host (tests of the error path)."""
    return _check(lib.pod_prefill_inject_error(), "pod_prefill_inject_error")


def pod_dense_decode_attn_static(kv, capacity: int, n_tokens: int, q, out, n_q_heads: int, n_kv_heads: int,
                                 head_dim: int, sm_scale: float = 0.0, stream: int = 0) -> int:
    """Decode attention over a caller-owned dense K/V buffer ``[2][n_kv_heads][capacity][head_dim]``
    for programs that cannot allocate device memory when they need attention (their pool owns the
    whole GPU, or an allocation's device-wide synchronisation is unaffordable): the split-K scratch
    is a fixed array inside the library.  Rows past ``n_tokens`` must hold finite numbers."""
    return _check(lib.pod_dense_decode_attn_static(_ptr(kv), capacity, n_tokens, _ptr(q), _ptr(out), n_q_heads,
                                                   n_kv_heads, head_dim, sm_scale, stream),
                  "pod_dense_decode_attn_static")


def pod_dense_decode_attn_static_status() -> int:
    """POD_ERR_DEVICE once if a kernel of the allocation-free entry gave up a bounded wait, else POD_OK."""
    return lib.pod_dense_decode_attn_static_status()


def pod_dense_decode_attn_static_inject_error() -> int:
    """Sets that error word from the host (tests of the error path)."""
    return _check(lib.pod_dense_decode_attn_static_inject_error(), "pod_dense_decode_attn_static_inject_error")
