"""ctypes binding of libcpattn: the same names as the C entry points, argument marshalling only.

Tensors are ``torch`` CUDA tensors (used for device memory and streams only); every step of the
path runs inside the library's kernels.  The shared library must have been built
(``python -m paper_2609_04774_b200.build``); loading fails loudly otherwise -- there is no
fallback path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcpattn.so")

CP_OK = 0
CP_ERR_INVALID_ARG, CP_ERR_UNSUPPORTED, CP_ERR_WORKSPACE, CP_ERR_CUDA, CP_ERR_TIMEOUT, CP_ERR_BOUNDS = -1, -2, -3, -4, -5, -6
CP_DTYPE_BF16, CP_DTYPE_F32 = 0, 1

EXPORTS = ["cp_strerror", "cp_last_error", "cp_ctx_create", "cp_ctx_destroy", "cp_ctx_poll_status", "cp_ctx_cache_schedule", "cp_ctx_selftest_wait_expiry", "cp_plan",
           "cp_workspace_bytes", "cp_schedule_inspect", "cp_prefill_attn", "cp_prefill_attn_batch", "cp_prefill_attn_shard", "cp_prefill_attn_chunk", "cp_prefill_attn_kvrange", "cp_prefill_attn_static", "cp_merge",
           "cp_kv_gather", "cp_kv_append", "cp_workspace_bytes_fp8", "cp_prefill_attn_fp8", "cp_prefill_attn_fp8_batch",
           "cp_kv_append_fp8", "cp_kv_append_segments", "cp_prefill_attn_fp8_shard", "cp_prefill_attn_fp8_chunk",
           "cp_prefill_attn_fp8_kvrange", "cp_kv_gather_fp8", "cp_kv_append_segments_fp8", "cp_check_page_table"]


class CpError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("%s (%d): %s" % (_strerror(code), code, message))
        self.code = code


class cp_shard_plan(ctypes.Structure):
    _fields_ = [("q_begin", ctypes.c_int64 * 2), ("q_end", ctypes.c_int64 * 2), ("kv_end", ctypes.c_int64 * 2),
                ("pairs", ctypes.c_uint64)]


class cp_kv_cache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("num_pages", ctypes.c_int64),
                ("page_size", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("stride_page", ctypes.c_int64), ("stride_tok", ctypes.c_int64),
                ("stride_head", ctypes.c_int64)]


class cp_kv_cache_fp8(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
                ("num_pages", ctypes.c_int64), ("page_size", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("stride_page", ctypes.c_int64), ("stride_tok", ctypes.c_int64),
                ("stride_head", ctypes.c_int64)]


_lib = None


def load():
    """Load libcpattn.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libcpattn.so is missing at %s: run `python -m paper_2609_04774_b200.build` "
                               "(there is no fallback implementation)" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        lib.cp_strerror.restype = ctypes.c_char_p
        lib.cp_strerror.argtypes = [ctypes.c_int]
        lib.cp_last_error.restype = ctypes.c_char_p
        lib.cp_workspace_bytes.restype = ctypes.c_size_t
        lib.cp_workspace_bytes_fp8.restype = ctypes.c_size_t
        for name in EXPORTS:
            if name not in ("cp_strerror", "cp_last_error", "cp_workspace_bytes", "cp_workspace_bytes_fp8"):
                getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _strerror(code: int) -> str:
    return load().cp_strerror(code).decode()


def _check(rc: int) -> None:
    if rc != CP_OK:
        raise CpError(rc, load().cp_last_error().decode())


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _hp(a):
    """Address of a host numpy array (the plain integer route; `ctypes.data_as` costs twice as much per call)."""
    return ctypes.c_void_p(a.ctypes.data)


def _stream(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class Context:
    """cp_ctx handle (cp_ctx_create / cp_ctx_destroy / cp_ctx_poll_status)."""

    def __init__(self, device: int = 0):
        self._h = ctypes.c_void_p()
        _check(load().cp_ctx_create(ctypes.byref(self._h), ctypes.c_int(device)))
        self.device = device

    def close(self):
        if self._h:
            load().cp_ctx_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def cache_schedule(self, enable: bool):
        """Reuse the work lists left in the workspace by the previous call when the next one has the same shape."""
        _check(load().cp_ctx_cache_schedule(self._h, ctypes.c_int(1 if enable else 0)))

    def selftest_wait_expiry(self, stream=None):
        """Enqueue the bounded-wait self-test; the next poll_status() after a sync raises CP_ERR_TIMEOUT."""
        _check(load().cp_ctx_selftest_wait_expiry(self._h, _stream(stream)))

    def poll_status(self):
        """Raises CpError if a device-side wait expired since the last poll."""
        detail = (ctypes.c_int32 * 4)()
        _check(load().cp_ctx_poll_status(self._h, detail))


def cp_plan(new_len: int, prefix_len: int, C: int):
    """Zigzag shard plan: list of C dicts {q_begin, q_end, kv_end, pairs}."""
    arr = (cp_shard_plan * max(C, 1))()
    _check(load().cp_plan(ctypes.c_int64(new_len), ctypes.c_int64(prefix_len), ctypes.c_int32(C), arr))
    return [{"q_begin": list(s.q_begin), "q_end": list(s.q_end), "kv_end": list(s.kv_end), "pairs": int(s.pairs)}
            for s in arr[:C]]


def cp_workspace_bytes(new_len, C, Hq) -> int:
    nl, cs = _i64(new_len).reshape(-1), _i32(C).reshape(-1)
    return int(load().cp_workspace_bytes(ctypes.c_int32(nl.size), _hp(nl),
                                         _hp(cs), ctypes.c_int32(Hq)))


def cp_schedule_inspect(cu_new, prefix_len, C, Hq, Hkv, num_sms=148, want_lists=True):
    """Host-only view of the varlen tile schedule: (summary dict, pieces [n,6] int32, items [n,4] int32)."""
    cu_new, prefix_len, C = _i64(cu_new), _i64(prefix_len), _i32(C)
    B = prefix_len.size
    summary = np.zeros(10, dtype=np.int64)
    args = [ctypes.c_int32(B), _hp(cu_new), _hp(prefix_len),
            _hp(C), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(num_sms),
            _hp(summary)]
    _check(load().cp_schedule_inspect(*args, None, ctypes.c_int64(0), None, ctypes.c_int64(0)))
    keys = ["grid", "tiles", "pieces", "split_units", "slots", "max_load", "min_load", "total", "inline", "launches"]
    info = dict(zip(keys, (int(x) for x in summary)))
    if not want_lists:
        return info, None, None
    pieces = np.zeros((info["pieces"], 6), dtype=np.int32)
    items = np.zeros((info["tiles"], 4), dtype=np.int32)
    _check(load().cp_schedule_inspect(*args, _hp(pieces), ctypes.c_int64(pieces.shape[0]),
                                      _hp(items), ctypes.c_int64(items.shape[0])))
    return info, pieces, items


def make_cache(k_pages, v_pages) -> cp_kv_cache:
    """Describe paged K/V tensors [num_pages, page_size, Hkv, D] (bf16, any strides with dim stride 1)."""
    assert k_pages.dim() == 4 and k_pages.stride() == v_pages.stride() and k_pages.stride(3) == 1
    c = cp_kv_cache()
    c.k, c.v = k_pages.data_ptr(), v_pages.data_ptr()
    c.num_pages, c.page_size, c.Hkv, c.D = k_pages.shape
    c.stride_page, c.stride_tok, c.stride_head = k_pages.stride(0), k_pages.stride(1), k_pages.stride(2)
    return c


def cp_prefill_attn(ctx, q, cache, page_table, prefix_len, new_len, C, Hq, scale, out, lse, workspace, stream=None):
    _check(load().cp_prefill_attn(ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len),
                                  ctypes.c_int64(new_len), ctypes.c_int32(C), ctypes.c_int32(Hq),
                                  ctypes.c_float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                  ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_batch(ctx, q, cache, page_table, cu_new, prefix_len, C, cu_pages, Hq, scale, out, lse, workspace,
                          stream=None):
    cu_new, prefix_len, cu_pages, C = _i64(cu_new), _i64(prefix_len), _i64(cu_pages), _i32(C)
    B = prefix_len.size
    assert cu_new.size == B + 1 and cu_pages.size == B + 1 and C.size == B
    _check(load().cp_prefill_attn_batch(
        ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int32(B),
        _hp(cu_new), _hp(prefix_len),
        _hp(C), _hp(cu_pages), ctypes.c_int32(Hq),
        ctypes.c_float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_shard(ctx, q, cache, page_table, prefix_len, new_len, C, shard, Hq, scale, partial_out,
                          partial_lse, workspace, stream=None):
    _check(load().cp_prefill_attn_shard(
        ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len), ctypes.c_int64(new_len),
        ctypes.c_int32(C), ctypes.c_int32(shard), ctypes.c_int32(Hq), ctypes.c_float(scale), _ptr(partial_out),
        _ptr(partial_lse), _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
        _stream(stream)))


def cp_prefill_attn_chunk(ctx, q_chunk, cache, page_table, prefix_len, new_len, C, chunk, Hq, scale, out_chunk,
                          lse_chunk, workspace, stream=None):
    """One zigzag chunk in chunk-local buffers: q_chunk/out_chunk [n,Hq,D] bf16, lse_chunk [Hq,n] fp32."""
    _check(load().cp_prefill_attn_chunk(
        ctx._h, _ptr(q_chunk), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len),
        ctypes.c_int64(new_len), ctypes.c_int32(C), ctypes.c_int32(chunk), ctypes.c_int32(Hq), ctypes.c_float(scale),
        _ptr(out_chunk), _ptr(lse_chunk), _ptr(workspace),
        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_kvrange(ctx, q, cache, page_table, prefix_len, new_len, kv_lo, kv_hi, Hq, scale, partial_out,
                            partial_lse, workspace, stream=None):
    """All R queries against keys at absolute positions [kv_lo, kv_hi) only: fp32 partial + LSE for cp_merge."""
    _check(load().cp_prefill_attn_kvrange(
        ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len), ctypes.c_int64(new_len),
        ctypes.c_int64(kv_lo), ctypes.c_int64(kv_hi), ctypes.c_int32(Hq), ctypes.c_float(scale), _ptr(partial_out),
        _ptr(partial_lse), _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
        _stream(stream)))


def cp_prefill_attn_static(q, cache, page_table, prefix_len, new_len, C, Hq, scale, out, lse, stream=None):
    """cp_prefill_attn without a context or a workspace: the library's built-in device scratch holds the
    tile list, so nothing is allocated.  For callers that cannot allocate device memory (all of HBM
    already handed to a cache pool, allocation-free serving loops).  Limits: ceil(new_len/128) + 2*C <= 2048
    tiles; calls share the scratch, so calls that may overlap on the GPU must be ordered by the caller."""
    _check(load().cp_prefill_attn_static(_ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len),
                                         ctypes.c_int64(new_len), ctypes.c_int32(C), ctypes.c_int32(Hq),
                                         ctypes.c_float(scale), _ptr(out), _ptr(lse), _stream(stream)))


def cp_merge(ctx, partials, lses, out, lse_out=None, stream=None):
    """partials [N,T,H,D] fp32, lses [N,H,T] fp32 -> out [T,H,D] (bf16 or fp32), lse_out [H,T] or None."""
    import torch
    N, T, H, D = partials.shape
    dt = CP_DTYPE_BF16 if out.dtype == torch.bfloat16 else CP_DTYPE_F32
    _check(load().cp_merge(ctx._h, _ptr(partials), _ptr(lses), ctypes.c_int32(N), ctypes.c_int64(T),
                           ctypes.c_int32(H), ctypes.c_int32(D), _ptr(out), ctypes.c_int32(dt), _ptr(lse_out),
                           _stream(stream)))


def cp_kv_gather(ctx, cache, page_table, t_begin, n, k_rows, v_rows, stream=None):
    _check(load().cp_kv_gather(ctx._h, ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(t_begin),
                               ctypes.c_int64(n), _ptr(k_rows), _ptr(v_rows), _stream(stream)))


def cp_kv_append(ctx, cache, page_table, t_begin, n, k_rows, v_rows, stream=None):
    _check(load().cp_kv_append(ctx._h, ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(t_begin),
                               ctypes.c_int64(n), _ptr(k_rows), _ptr(v_rows), _stream(stream)))


def cp_kv_append_segments(ctx, cache, page_table, segments, k_rows, v_rows, stream=None):
    """segments: iterable of (t_begin, n, row0); rows [row0, row0+n) of k_rows / v_rows go to tokens [t_begin, t_begin+n)."""
    seg = np.ascontiguousarray(np.asarray(list(segments), dtype=np.int64).reshape(-1, 3))
    _check(load().cp_kv_append_segments(ctx._h, ctypes.byref(cache), _ptr(page_table), ctypes.c_int32(seg.shape[0]),
                                        _hp(seg), _ptr(k_rows), _ptr(v_rows), _stream(stream)))


# ------------------------------------------------------------------------------------------------
# FP8 K/V variant
# ------------------------------------------------------------------------------------------------

def make_cache_fp8(k8_pages, v8_pages, k_scale, v_scale) -> cp_kv_cache_fp8:
    """Describe paged E4M3 K/V tensors [num_pages, page_size, Hkv, D] (uint8) with fp32 scales [Hkv] on the device."""
    assert k8_pages.dim() == 4 and k8_pages.stride() == v8_pages.stride() and k8_pages.stride(3) == 1
    assert k8_pages.element_size() == 1 and k_scale.numel() == k8_pages.shape[2] == v_scale.numel()
    c = cp_kv_cache_fp8()
    c.k, c.v, c.k_scale, c.v_scale = k8_pages.data_ptr(), v8_pages.data_ptr(), k_scale.data_ptr(), v_scale.data_ptr()
    c.num_pages, c.page_size, c.Hkv, c.D = k8_pages.shape
    c.stride_page, c.stride_tok, c.stride_head = k8_pages.stride(0), k8_pages.stride(1), k8_pages.stride(2)
    return c


def cp_workspace_bytes_fp8(new_len, C, Hq) -> int:
    nl, cs = _i64(new_len).reshape(-1), _i32(C).reshape(-1)
    return int(load().cp_workspace_bytes_fp8(ctypes.c_int32(nl.size), _hp(nl), _hp(cs), ctypes.c_int32(Hq)))


def cp_prefill_attn_fp8(ctx, q, cache, page_table, prefix_len, new_len, C, Hq, scale, out, lse, workspace, stream=None):
    _check(load().cp_prefill_attn_fp8(ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len),
                                      ctypes.c_int64(new_len), ctypes.c_int32(C), ctypes.c_int32(Hq),
                                      ctypes.c_float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                      ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_fp8_batch(ctx, q, cache, page_table, cu_new, prefix_len, C, cu_pages, Hq, scale, out, lse, workspace,
                              stream=None):
    cu_new, prefix_len, cu_pages, C = _i64(cu_new), _i64(prefix_len), _i64(cu_pages), _i32(C)
    B = prefix_len.size
    assert cu_new.size == B + 1 and cu_pages.size == B + 1 and C.size == B
    _check(load().cp_prefill_attn_fp8_batch(
        ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int32(B), _hp(cu_new), _hp(prefix_len), _hp(C),
        _hp(cu_pages), ctypes.c_int32(Hq), ctypes.c_float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_fp8_shard(ctx, q, cache, page_table, prefix_len, new_len, C, shard, Hq, scale, partial_out, partial_lse,
                              workspace, stream=None):
    _check(load().cp_prefill_attn_fp8_shard(
        ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len), ctypes.c_int64(new_len),
        ctypes.c_int32(C), ctypes.c_int32(shard), ctypes.c_int32(Hq), ctypes.c_float(scale), _ptr(partial_out),
        _ptr(partial_lse), _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_fp8_chunk(ctx, q_chunk, cache, page_table, prefix_len, new_len, C, chunk, Hq, scale, out_chunk, lse_chunk,
                              workspace, stream=None):
    _check(load().cp_prefill_attn_fp8_chunk(
        ctx._h, _ptr(q_chunk), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len), ctypes.c_int64(new_len),
        ctypes.c_int32(C), ctypes.c_int32(chunk), ctypes.c_int32(Hq), ctypes.c_float(scale), _ptr(out_chunk), _ptr(lse_chunk),
        _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_prefill_attn_fp8_kvrange(ctx, q, cache, page_table, prefix_len, new_len, kv_lo, kv_hi, Hq, scale, partial_out,
                                partial_lse, workspace, stream=None):
    _check(load().cp_prefill_attn_fp8_kvrange(
        ctx._h, _ptr(q), ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(prefix_len), ctypes.c_int64(new_len),
        ctypes.c_int64(kv_lo), ctypes.c_int64(kv_hi), ctypes.c_int32(Hq), ctypes.c_float(scale), _ptr(partial_out),
        _ptr(partial_lse), _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def cp_kv_append_fp8(ctx, cache, page_table, t_begin, n, k_rows, v_rows, stream=None):
    """bf16 rows [n, Hkv, D] -> E4M3 bytes of logical tokens t_begin.. of the FP8 cache (per-head scales)."""
    _check(load().cp_kv_append_fp8(ctx._h, ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(t_begin),
                                   ctypes.c_int64(n), _ptr(k_rows), _ptr(v_rows), _stream(stream)))


def cp_kv_gather_fp8(ctx, cache, page_table, t_begin, n, k_bytes, v_bytes, stream=None):
    """Raw E4M3 bytes of logical tokens [t_begin, t_begin + n) -> k_bytes / v_bytes [n, Hkv, D] uint8."""
    _check(load().cp_kv_gather_fp8(ctx._h, ctypes.byref(cache), _ptr(page_table), ctypes.c_int64(t_begin),
                                   ctypes.c_int64(n), _ptr(k_bytes), _ptr(v_bytes), _stream(stream)))


def cp_kv_append_segments_fp8(ctx, cache, page_table, segments, k_bytes, v_bytes, stream=None):
    """cp_kv_append_segments for an FP8 cache: rows of stored bytes, copied as they are."""
    seg = np.ascontiguousarray(np.asarray(list(segments), dtype=np.int64).reshape(-1, 3))
    _check(load().cp_kv_append_segments_fp8(ctx._h, ctypes.byref(cache), _ptr(page_table), ctypes.c_int32(seg.shape[0]),
                                            _hp(seg), _ptr(k_bytes), _ptr(v_bytes), _stream(stream)))


def cp_check_page_table(ctx, page_table, num_pages, stream=None):
    """Enqueue the page-table check; a bad entry shows as CP_ERR_BOUNDS at the next poll_status() after a sync."""
    _check(load().cp_check_page_table(ctx._h, _ptr(page_table), ctypes.c_int64(page_table.numel()),
                                      ctypes.c_int64(num_pages), _stream(stream)))
