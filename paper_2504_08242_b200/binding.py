"""Thin ctypes binding of libjupiter.so: argument marshalling only.

Every function has the name and argument order of its C entry point in
``include/jupiter.h``; tensors are torch CUDA tensors used purely as device
memory (``data_ptr()``) and the stream is torch's current stream unless given.
No arithmetic happens here and there is no fallback: if the library cannot be
loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

c_void_p, c_int32, c_int64, c_float, c_size_t = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                                 ctypes.c_float, ctypes.c_size_t)

STATUS_NAMES = {
    0: "JUPITER_OK", 1: "JUPITER_ERR_INVALID_ARG", 2: "JUPITER_ERR_OUT_OF_RANGE", 3: "JUPITER_ERR_UNSUPPORTED",
    4: "JUPITER_ERR_ALIGNMENT", 5: "JUPITER_ERR_WORKSPACE", 6: "JUPITER_ERR_CUDA", 7: "JUPITER_ERR_TIMEOUT",
}
BRANCH_AUTO, BRANCH_STREAM, BRANCH_SPLIT_KV, BRANCH_TENSOR_CORE = range(4)
(OK, ERR_INVALID_ARG, ERR_OUT_OF_RANGE, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA,
 ERR_TIMEOUT) = range(8)

EXPORTS = (
    "jupiter_create", "jupiter_destroy", "jupiter_status_string", "jupiter_last_cuda_error",
    "jupiter_poll_device_status", "jupiter_launch_count", "jupiter_kv_append",
    "jupiter_chunk_prefill_attn", "jupiter_branch_attn", "jupiter_branch_attn_noalloc",
    "jupiter_plan_sequence_partition", "jupiter_branch_attn_tree", "jupiter_branch_prefill_attn",
    "jupiter_chunk_prefill_append_attn", "jupiter_branch_append_attn", "jupiter_read_probe",
    "jupiter_kv_compact", "jupiter_wait_probe", "jupiter_select_branch_kernel",
    "jupiter_branch_append_attn_layers",
)


class jupiter_kv_cache(ctypes.Structure):
    _fields_ = [("k", c_void_p), ("v", c_void_p), ("batch", c_int32), ("kv_heads", c_int32),
                ("capacity", c_int32), ("head_dim", c_int32), ("stride_batch", c_int64),
                ("stride_head", c_int64), ("stride_row", c_int64)]


class jupiter_branch_layer(ctypes.Structure):
    _fields_ = [("q", c_void_p), ("k_new", c_void_p), ("v_new", c_void_p), ("prefix", ctypes.POINTER(jupiter_kv_cache)),
                ("suffix", ctypes.POINTER(jupiter_kv_cache)), ("out", c_void_p), ("lse", c_void_p)]


class JupiterError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        super().__init__(f"{STATUS_NAMES.get(status, status)}" + (f": {detail}" if detail else ""))


def library_path() -> str:
    return _build.LIB


def _load() -> ctypes.CDLL:
    path = library_path()
    if _build.is_stale():
        _build.build()  # raises if nvcc is missing; there is no other implementation to fall back to
    lib = ctypes.CDLL(path)
    P = ctypes.POINTER
    lib.jupiter_create.argtypes = [P(c_void_p), ctypes.c_int, c_size_t]
    lib.jupiter_create.restype = ctypes.c_int
    lib.jupiter_destroy.argtypes = [c_void_p]
    lib.jupiter_destroy.restype = None
    lib.jupiter_status_string.argtypes = [ctypes.c_int]
    lib.jupiter_status_string.restype = ctypes.c_char_p
    lib.jupiter_last_cuda_error.argtypes = [c_void_p]
    lib.jupiter_last_cuda_error.restype = ctypes.c_char_p
    lib.jupiter_poll_device_status.argtypes = [c_void_p, c_void_p]
    lib.jupiter_poll_device_status.restype = ctypes.c_int
    lib.jupiter_launch_count.argtypes = [c_void_p]
    lib.jupiter_launch_count.restype = ctypes.c_uint64
    lib.jupiter_kv_compact.argtypes = [c_void_p, P(jupiter_kv_cache), c_int32, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.jupiter_kv_compact.restype = ctypes.c_int
    lib.jupiter_branch_append_attn_layers.argtypes = [c_void_p, P(jupiter_branch_layer), c_int32, c_int32, c_void_p,
                                                      c_int32, c_int32, c_int32, c_int32, c_float, c_void_p]
    lib.jupiter_branch_append_attn_layers.restype = ctypes.c_int
    lib.jupiter_select_branch_kernel.argtypes = [c_void_p, ctypes.c_int]
    lib.jupiter_select_branch_kernel.restype = ctypes.c_int
    lib.jupiter_wait_probe.argtypes = [c_void_p, c_int64, c_void_p]
    lib.jupiter_wait_probe.restype = ctypes.c_int
    lib.jupiter_read_probe.argtypes = [c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.jupiter_read_probe.restype = ctypes.c_int
    lib.jupiter_kv_append.argtypes = [c_void_p, P(jupiter_kv_cache), c_void_p, c_void_p, c_int32, c_int32,
                                      c_void_p, c_void_p]
    lib.jupiter_kv_append.restype = ctypes.c_int
    lib.jupiter_chunk_prefill_attn.argtypes = [c_void_p, c_void_p, P(jupiter_kv_cache), c_int32, c_int32, c_int32,
                                               c_float, c_void_p, c_void_p, c_void_p]
    lib.jupiter_chunk_prefill_attn.restype = ctypes.c_int
    lib.jupiter_chunk_prefill_append_attn.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, P(jupiter_kv_cache),
                                                      c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p]
    lib.jupiter_chunk_prefill_append_attn.restype = ctypes.c_int
    lib.jupiter_branch_attn.argtypes = [c_void_p, c_void_p, P(jupiter_kv_cache), c_int32, P(jupiter_kv_cache),
                                        c_void_p, c_int32, c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p,
                                        c_void_p]
    lib.jupiter_branch_attn.restype = ctypes.c_int
    lib.jupiter_branch_append_attn.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, P(jupiter_kv_cache), c_int32,
                                               P(jupiter_kv_cache), c_void_p, c_int32, c_int32, c_int32, c_int32,
                                               c_float, c_void_p, c_void_p, c_void_p]
    lib.jupiter_branch_append_attn.restype = ctypes.c_int
    lib.jupiter_branch_attn_noalloc.argtypes = lib.jupiter_branch_attn.argtypes[1:]
    lib.jupiter_branch_attn_noalloc.restype = ctypes.c_int
    lib.jupiter_branch_prefill_attn.argtypes = [c_void_p, c_void_p, P(jupiter_kv_cache), c_int32, P(jupiter_kv_cache),
                                                c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p]
    lib.jupiter_branch_prefill_attn.restype = ctypes.c_int
    lib.jupiter_branch_attn_tree.argtypes = [c_void_p, c_void_p, P(jupiter_kv_cache), c_int32, P(jupiter_kv_cache),
                                             c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_float, c_void_p,
                                             c_void_p, c_void_p]
    lib.jupiter_branch_attn_tree.restype = ctypes.c_int
    lib.jupiter_plan_sequence_partition.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_int32, c_int32,
                                                    c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                                    c_void_p]
    lib.jupiter_plan_sequence_partition.restype = ctypes.c_int
    return lib


lib = _load()


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def cache_desc(k: torch.Tensor, v: torch.Tensor) -> jupiter_kv_cache:
    """Descriptor of a head-major cache held in two bf16 tensors [batch][kv_heads][capacity][D]."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 4
    assert k.shape == v.shape and k.stride() == v.stride() and k.stride(3) == 1
    B, H, cap, D = k.shape
    return jupiter_kv_cache(k.data_ptr(), v.data_ptr(), B, H, cap, D, k.stride(0), k.stride(1), k.stride(2))


class Context:
    """Owns a jupiter_ctx.  Methods mirror the C entry points and raise JupiterError on a non-OK status."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        h = c_void_p()
        st = lib.jupiter_create(ctypes.byref(h), int(device), int(workspace_bytes))
        if st != OK:
            raise JupiterError(st, "jupiter_create")
        self._h = h
        self.device = device

    def close(self):
        if getattr(self, "_h", None):
            lib.jupiter_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != OK:
            detail = lib.jupiter_last_cuda_error(self._h).decode() if st == ERR_CUDA else ""
            raise JupiterError(st, detail)

    def launch_count(self) -> int:
        return int(lib.jupiter_launch_count(self._h))

    def kv_compact(self, cache: jupiter_kv_cache, q_len: int, d_pos, d_accept, d_n_accept, stream=None):
        self._check(lib.jupiter_kv_compact(self._h, ctypes.byref(cache), q_len, _ptr(d_pos), _ptr(d_accept),
                                           _ptr(d_n_accept), _stream(stream)))

    def read_probe(self, src, nbytes: int, out, stream=None):
        self._check(lib.jupiter_read_probe(self._h, _ptr(src), nbytes, _ptr(out), _stream(stream)))

    def select_branch_kernel(self, which: int):
        self._check(lib.jupiter_select_branch_kernel(self._h, int(which)))

    def wait_probe(self, limit_cycles: int, stream=None):
        self._check(lib.jupiter_wait_probe(self._h, int(limit_cycles), _stream(stream)))

    def poll_device_status(self, stream=None) -> int:
        return int(lib.jupiter_poll_device_status(self._h, _stream(stream)))

    def kv_append(self, cache: jupiter_kv_cache, k_new, v_new, n_rows: int, pos: int = 0, d_pos=None, stream=None):
        self._check(lib.jupiter_kv_append(self._h, ctypes.byref(cache), _ptr(k_new), _ptr(v_new), n_rows, pos,
                                          _ptr(d_pos), _stream(stream)))

    def chunk_prefill_attn(self, q, cache: jupiter_kv_cache, q_heads: int, q_len: int, pos: int, scale: float,
                           out, lse=None, stream=None):
        self._check(lib.jupiter_chunk_prefill_attn(self._h, _ptr(q), ctypes.byref(cache), q_heads, q_len, pos,
                                                   scale, _ptr(out), _ptr(lse), _stream(stream)))

    def chunk_prefill_append_attn(self, q, k_new, v_new, cache: jupiter_kv_cache, q_heads: int, q_len: int, pos: int,
                                  scale: float, out, lse=None, stream=None):
        self._check(lib.jupiter_chunk_prefill_append_attn(self._h, _ptr(q), _ptr(k_new), _ptr(v_new),
                                                          ctypes.byref(cache), q_heads, q_len, pos, scale, _ptr(out),
                                                          _ptr(lse), _stream(stream)))

    def branch_attn(self, q, prefix: jupiter_kv_cache, prefix_len: int, suffix: jupiter_kv_cache, d_suffix_len,
                    max_suffix_len: int, n_branches: int, q_heads: int, q_len: int, scale: float, out, lse=None,
                    stream=None):
        pfx = ctypes.byref(prefix) if prefix is not None else None
        self._check(lib.jupiter_branch_attn(self._h, _ptr(q), pfx, prefix_len, ctypes.byref(suffix),
                                            _ptr(d_suffix_len), max_suffix_len, n_branches, q_heads, q_len, scale,
                                            _ptr(out), _ptr(lse), _stream(stream)))

    def branch_append_attn(self, q, k_new, v_new, prefix: jupiter_kv_cache, prefix_len: int, suffix: jupiter_kv_cache,
                           d_suffix_len, max_suffix_len: int, n_branches: int, q_heads: int, q_len: int, scale: float,
                           out, lse=None, stream=None):
        pfx = ctypes.byref(prefix) if prefix is not None else None
        self._check(lib.jupiter_branch_append_attn(self._h, _ptr(q), _ptr(k_new), _ptr(v_new), pfx, prefix_len,
                                                   ctypes.byref(suffix), _ptr(d_suffix_len), max_suffix_len,
                                                   n_branches, q_heads, q_len, scale, _ptr(out), _ptr(lse),
                                                   _stream(stream)))

    def branch_append_attn_layers(self, layers, prefix_len: int, d_suffix_len, max_suffix_len: int, n_branches: int,
                                  q_heads: int, q_len: int, scale: float, stream=None):
        """layers: sequence of (q, k_new, v_new, prefix descriptor or None, suffix descriptor, out, lse or None)."""
        arr = (jupiter_branch_layer * len(layers))()
        for i, (q, kn, vn, pfx, sfx, out, lse) in enumerate(layers):
            arr[i].q, arr[i].k_new, arr[i].v_new = q.data_ptr(), kn.data_ptr(), vn.data_ptr()
            arr[i].prefix = ctypes.pointer(pfx) if pfx is not None else None
            arr[i].suffix = ctypes.pointer(sfx)
            arr[i].out = out.data_ptr()
            arr[i].lse = lse.data_ptr() if lse is not None else None
        self._check(lib.jupiter_branch_append_attn_layers(self._h, arr, len(layers), prefix_len, _ptr(d_suffix_len),
                                                          max_suffix_len, n_branches, q_heads, q_len, scale,
                                                          _stream(stream)))

    def branch_prefill_attn(self, q, prefix: jupiter_kv_cache, prefix_len: int, cache: jupiter_kv_cache,
                            q_heads: int, q_len: int, pos: int, scale: float, out, lse=None, stream=None):
        pfx = ctypes.byref(prefix) if prefix is not None else None
        self._check(lib.jupiter_branch_prefill_attn(self._h, _ptr(q), pfx, prefix_len, ctypes.byref(cache), q_heads,
                                                    q_len, pos, scale, _ptr(out), _ptr(lse), _stream(stream)))

    def branch_attn_tree(self, q, prefix: jupiter_kv_cache, prefix_len: int, suffix: jupiter_kv_cache, d_suffix_len,
                         d_tree_mask, max_suffix_len: int, n_branches: int, q_heads: int, q_len: int, scale: float,
                         out, lse=None, stream=None):
        pfx = ctypes.byref(prefix) if prefix is not None else None
        self._check(lib.jupiter_branch_attn_tree(self._h, _ptr(q), pfx, prefix_len, ctypes.byref(suffix),
                                                 _ptr(d_suffix_len), _ptr(d_tree_mask), max_suffix_len, n_branches,
                                                 q_heads, q_len, scale, _ptr(out), _ptr(lse), _stream(stream)))


def branch_attn_noalloc(q, prefix: jupiter_kv_cache, prefix_len: int, suffix: jupiter_kv_cache, d_suffix_len,
                        max_suffix_len: int, n_branches: int, q_heads: int, q_len: int, scale: float, out, lse=None,
                        stream=None):
    """jupiter_branch_attn_noalloc: same as Context.branch_attn but with no context and no allocation --
    the split-KV scratch is a fixed array inside the library.  Runs on the current CUDA device."""
    pfx = ctypes.byref(prefix) if prefix is not None else None
    st = lib.jupiter_branch_attn_noalloc(_ptr(q), pfx, prefix_len, ctypes.byref(suffix), _ptr(d_suffix_len),
                                         max_suffix_len, n_branches, q_heads, q_len, scale, _ptr(out), _ptr(lse),
                                         _stream(stream))
    if st != OK:
        raise JupiterError(st, "jupiter_branch_attn_noalloc")


def plan_sequence_partition(q_table, xs, ys, seq_len: int, min_len: int, max_parts: int, n_stages: int,
                            granularity: int = 1):
    """jupiter_plan_sequence_partition on host arrays (numpy): q_table [len(xs)][len(ys)] float32.
    Returns (k, lengths, slowest, latency)."""
    import numpy as np
    q = np.ascontiguousarray(q_table, dtype=np.float32)
    gx = np.ascontiguousarray(xs, dtype=np.int32)
    gy = np.ascontiguousarray(ys, dtype=np.int32)
    assert q.shape == (gx.size, gy.size)
    k = ctypes.c_int32(0)
    lengths = np.zeros(max(max_parts, 1), np.int32)
    slowest, latency = ctypes.c_float(0), ctypes.c_float(0)
    st = lib.jupiter_plan_sequence_partition(q.ctypes.data, gx.ctypes.data, gx.size, gy.ctypes.data, gy.size,
                                             seq_len, min_len, max_parts, n_stages, granularity, ctypes.addressof(k),
                                             lengths.ctypes.data, ctypes.addressof(slowest),
                                             ctypes.addressof(latency))
    if st != OK:
        raise JupiterError(st, "jupiter_plan_sequence_partition")
    return int(k.value), lengths[:k.value].tolist(), float(slowest.value), float(latency.value)
