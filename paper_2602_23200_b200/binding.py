"""ctypes binding over libinnerq.so: argument marshalling only.

Function names mirror the C ABI (include/innerq.h).  PyTorch is used for device memory and
streams; every step of the path runs in the library's CUDA kernels.  There is no CPU fallback:
if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libinnerq.so")

MODE_SYM, MODE_ASYM, MODE_HYBRID = 0, 1, 2
SYM_FULLRANGE, SYM_PAPER_LITERAL = 0, 1
GROUPING_INNER, GROUPING_OUTER, GROUPING_FP16 = 0, 1, 2

EXPORTED_SYMBOLS = (
    "innerq_cache_bytes", "innerq_token_payload_bytes", "innerq_cache_create", "innerq_cache_destroy",
    "innerq_cache_n_tokens", "innerq_quantize_prefill", "innerq_append_token", "innerq_decode_attention",
    "innerq_decode_attention_static", "innerq_decode_step_host", "innerq_step_staging_bytes",
    "innerq_decode_attention_multi", "innerq_multi_query_scratch_bytes",
    "innerq_append_token_batched", "innerq_decode_attention_batched",
    "innerq_paged_cache_bytes", "innerq_cache_create_paged", "innerq_cache_pages_for", "innerq_cache_pages_assigned",
    "innerq_cache_assign_pages", "innerq_cache_release_pages",
    "innerq_cache_export", "innerq_cache_import", "innerq_set_decode_options", "innerq_last_launch_count", "innerq_read_device_error",
    "innerq_selftest_wait_expiry", "innerq_status_string",
)


class InnerQError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


class innerq_config_t(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "max_tokens", "group", "k_bits", "v_bits",
        "k_mode", "v_mode", "sym_variant", "w_sink", "w_recent", "grouping", "k_normalize")] + [("sm_scale", C.c_float)]


class innerq_export_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "k_code", "v_code", "k_scale", "k_zero", "v_scale", "v_zero", "norm",
        "k_sink", "v_sink", "k_recent", "v_recent")] + [(n, C.c_int32) for n in (
        "n_tokens", "n_sink", "n_qk", "n_qv", "n_k_recent", "n_v_recent")]


_lib = None


def lib() -> C.CDLL:
    """Load libinnerq.so (built in-tree by paper_2602_23200_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_23200_b200.build` "
                           "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    cfgp = C.POINTER(innerq_config_t)
    L.innerq_cache_bytes.argtypes = [cfgp, C.POINTER(sz), C.POINTER(sz)]
    L.innerq_token_payload_bytes.argtypes = [cfgp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.innerq_cache_create.argtypes = [cfgp, vp, sz, vp, sz, vp, C.POINTER(vp)]
    L.innerq_cache_destroy.argtypes = [vp]
    L.innerq_cache_n_tokens.argtypes = [vp]
    L.innerq_quantize_prefill.argtypes = [vp, vp, vp, i32, vp]
    L.innerq_append_token.argtypes = [vp, vp, vp, vp]
    L.innerq_decode_attention.argtypes = [vp, vp, vp, vp]
    L.innerq_decode_attention_static.argtypes = [vp, vp, vp, vp]
    L.innerq_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.innerq_step_staging_bytes.argtypes = [cfgp, C.POINTER(sz)]
    L.innerq_decode_attention_multi.argtypes = [vp, vp, vp, i32, vp, sz, vp]
    L.innerq_multi_query_scratch_bytes.argtypes = [cfgp, C.POINTER(sz)]
    L.innerq_append_token_batched.argtypes = [C.POINTER(vp), i32, vp, vp, vp]
    L.innerq_decode_attention_batched.argtypes = [C.POINTER(vp), i32, vp, vp, vp]
    L.innerq_paged_cache_bytes.argtypes = [cfgp, i32, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz), C.POINTER(i32)]
    L.innerq_cache_create_paged.argtypes = [cfgp, i32, vp, sz, vp, sz, vp, i32, vp, C.POINTER(vp)]
    L.innerq_cache_pages_for.argtypes = [vp, i32]
    L.innerq_cache_pages_assigned.argtypes = [vp]
    L.innerq_cache_assign_pages.argtypes = [vp, C.POINTER(i32), i32, vp]
    L.innerq_cache_release_pages.argtypes = [vp, C.POINTER(i32), i32]
    L.innerq_cache_export.argtypes = [vp, C.POINTER(innerq_export_t), vp]
    L.innerq_cache_import.argtypes = [vp, C.POINTER(innerq_export_t), C.c_int32, vp]
    L.innerq_set_decode_options.argtypes = [vp, i32, i32]
    L.innerq_last_launch_count.argtypes = [vp, i32]
    L.innerq_read_device_error.argtypes = [vp, vp]
    L.innerq_selftest_wait_expiry.argtypes = [vp, vp]
    L.innerq_status_string.argtypes = [C.c_int]
    L.innerq_status_string.restype = C.c_char_p
    for name in EXPORTED_SYMBOLS:
        if name != "innerq_status_string":
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().innerq_status_string(int(status)).decode()


def _check(status: int, what: str) -> int:
    if status < 0:
        raise InnerQError(status, what)
    return status


def make_config(w=None, **kw) -> innerq_config_t:
    """Build an innerq_config_t from a workload-like object (attribute names of synth.Workload) and/or keywords."""
    vals = dict(batch=1, n_q_heads=1, n_kv_heads=1, head_dim=128, max_tokens=0, group=32, k_bits=2, v_bits=2,
                k_mode=MODE_HYBRID, v_mode=MODE_HYBRID, sym_variant=0, w_sink=4, w_recent=128,
                grouping=GROUPING_INNER, k_normalize=1, sm_scale=0.0)
    if w is not None:
        for k in vals:
            if hasattr(w, k):
                vals[k] = getattr(w, k)
        if not kw.get("max_tokens") and hasattr(w, "n_tokens"):
            vals["max_tokens"] = w.n_tokens
    vals.update(kw)
    cfg = innerq_config_t()
    for k, v in vals.items():
        setattr(cfg, k, v)
    return cfg


def innerq_cache_bytes(cfg: innerq_config_t):
    cb, wb = C.c_size_t(), C.c_size_t()
    _check(lib().innerq_cache_bytes(C.byref(cfg), C.byref(cb), C.byref(wb)), "innerq_cache_bytes")
    return cb.value, wb.value


def innerq_token_payload_bytes(cfg: innerq_config_t):
    kb, vb = C.c_double(), C.c_double()
    _check(lib().innerq_token_payload_bytes(C.byref(cfg), C.byref(kb), C.byref(vb)), "innerq_token_payload_bytes")
    return kb.value, vb.value


def innerq_paged_cache_bytes(cfg: innerq_config_t, page_tokens: int):
    """(cache_bytes, workspace_bytes, page_bytes, max_pages) of a paged cache."""
    cb, wb, pb, mp = C.c_size_t(), C.c_size_t(), C.c_size_t(), C.c_int32()
    _check(lib().innerq_paged_cache_bytes(C.byref(cfg), int(page_tokens), C.byref(cb), C.byref(wb), C.byref(pb), C.byref(mp)),
           "innerq_paged_cache_bytes")
    return cb.value, wb.value, pb.value, mp.value


class PagePool:
    """A pool of cache pages in one torch device buffer, with the free list a caller of the C ABI keeps itself.
    `order` (a permutation of range(n_pages)) sets the order in which free pages are handed out."""

    def __init__(self, cfg: innerq_config_t, page_tokens: int, n_pages: int, device=None, order=None):
        import torch
        self.cfg, self.page_tokens, self.n_pages = cfg, int(page_tokens), int(n_pages)
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.page_bytes = innerq_paged_cache_bytes(cfg, page_tokens)[2]
        self.buf = torch.empty(self.n_pages * self.page_bytes, dtype=torch.uint8, device=self.device)
        self.free = list(range(self.n_pages)) if order is None else [int(i) for i in order]
        if sorted(self.free) != list(range(self.n_pages)):
            raise ValueError("order must be a permutation of range(n_pages)")

    def take(self, n: int):
        if n > len(self.free):
            raise RuntimeError(f"page pool exhausted: {n} pages wanted, {len(self.free)} free")
        out, self.free = self.free[:n], self.free[n:]
        return out

    def give_back(self, pages):
        self.free.extend(int(i) for i in pages)


def _stream_ptr(stream, device=None) -> int:
    """Raw cudaStream_t of `stream` (default: the current stream).  The library launches on the CURRENT device,
    so a call for a cache that lives on another device is refused here instead of faulting on the GPU."""
    import torch
    if device is not None and torch.cuda.current_device() != device.index:
        raise RuntimeError(f"the current CUDA device is {torch.cuda.current_device()}, the cache lives on {device}: "
                           "make the cache's device current (torch.cuda.set_device / torch.cuda.device) for the call")
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _dev_ptr(t, name: str, shape, device=None) -> int:
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float16 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA fp16 tensor")
    if device is not None and t.device != device:
        raise ValueError(f"{name} is on {t.device}, the cache on {device}")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")
    return t.data_ptr()


def _handles(caches):
    if not caches or any(not isinstance(c, InnerQCache) for c in caches):
        raise TypeError("caches must be a non-empty sequence of InnerQCache objects")
    arr = (C.c_void_p * len(caches))(*[c._h for c in caches])
    return arr


def innerq_append_token_batched(caches, k_new, v_new, stream=None):
    """Appends one token to every cache of the list (same configuration, own lengths): k_new, v_new are
    fp16 [n, batch, n_kv_heads, head_dim] device tensors, row i for caches[i]."""
    c = caches[0].cfg
    shape = (len(caches), c.batch, c.n_kv_heads, c.head_dim)
    _check(lib().innerq_append_token_batched(_handles(caches), len(caches), _dev_ptr(k_new, "k_new", shape, caches[0].device),
                                             _dev_ptr(v_new, "v_new", shape, caches[0].device), _stream_ptr(stream, caches[0].device)),
           "innerq_append_token_batched")


def innerq_decode_attention_batched(caches, q, out=None, stream=None):
    """Decode attention for every cache of the list over its own tokens: q fp16 [n, batch, n_q_heads, head_dim]."""
    import torch
    c = caches[0].cfg
    shape = (len(caches), c.batch, c.n_q_heads, c.head_dim)
    if out is None:
        out = torch.empty(shape, dtype=torch.float16, device=caches[0].device)
    _check(lib().innerq_decode_attention_batched(_handles(caches), len(caches), _dev_ptr(q, "q", shape, caches[0].device),
                                                 _dev_ptr(out, "out", shape, caches[0].device), _stream_ptr(stream, caches[0].device)),
           "innerq_decode_attention_batched")
    return out


class InnerQCache:
    """A packed KV cache living in caller-side torch device buffers, driven through the C ABI."""

    def __init__(self, cfg: innerq_config_t, device=None, stream=None, pool: "PagePool | None" = None):
        """pool: keep the packed part of the cache in pages of this pool (innerq_cache_create_paged) instead of inside
        the cache's own buffer; pages are assigned with ensure_pages / innerq_cache_assign_pages."""
        import torch
        self.cfg = cfg
        self.pool = pool
        # default: the current device (one process per GPU sets it once with torch.cuda.set_device)
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        if self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        if pool is not None and pool.device != self.device:
            raise ValueError(f"the pool is on {pool.device}, the cache on {self.device}")
        cb, wb = innerq_cache_bytes(cfg) if pool is None else innerq_paged_cache_bytes(cfg, pool.page_tokens)[:2]
        self.cache_bytes, self.workspace_bytes = cb, wb
        with torch.cuda.device(self.device):
            self._cache_buf = torch.empty(cb, dtype=torch.uint8, device=self.device)
            self._ws_buf = torch.empty(wb, dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            if pool is None:
                _check(lib().innerq_cache_create(C.byref(cfg), self._cache_buf.data_ptr(), cb, self._ws_buf.data_ptr(), wb,
                                                 _stream_ptr(stream, self.device), C.byref(h)), "innerq_cache_create")
            else:
                _check(lib().innerq_cache_create_paged(C.byref(cfg), pool.page_tokens, self._cache_buf.data_ptr(), cb,
                                                       self._ws_buf.data_ptr(), wb, pool.buf.data_ptr(), pool.n_pages,
                                                       _stream_ptr(stream, self.device), C.byref(h)),
                       "innerq_cache_create_paged")
        self._h = h

    # ---- paged caches
    def innerq_cache_pages_for(self, n_tokens: int) -> int:
        return _check(lib().innerq_cache_pages_for(self._h, int(n_tokens)), "innerq_cache_pages_for")

    @property
    def pages_assigned(self) -> int:
        return _check(lib().innerq_cache_pages_assigned(self._h), "innerq_cache_pages_assigned")

    def innerq_cache_assign_pages(self, pages, stream=None):
        arr = (C.c_int32 * len(pages))(*[int(i) for i in pages])
        _check(lib().innerq_cache_assign_pages(self._h, arr, len(pages), _stream_ptr(stream, self.device)),
               "innerq_cache_assign_pages")

    def innerq_cache_release_pages(self):
        """Empties the cache and returns the pool indices of the pages it held."""
        n = self.pages_assigned
        arr = (C.c_int32 * max(n, 1))()
        got = _check(lib().innerq_cache_release_pages(self._h, arr, n), "innerq_cache_release_pages")
        return [int(arr[i]) for i in range(got)]

    def ensure_pages(self, n_tokens: int, stream=None):
        """Takes from the pool's free list whatever the cache still lacks to hold n_tokens tokens."""
        if self.pool is None:
            return
        lack = self.innerq_cache_pages_for(n_tokens) - self.pages_assigned
        if lack > 0:
            self.innerq_cache_assign_pages(self.pool.take(lack), stream)

    def release_to_pool(self):
        if self.pool is not None:
            self.pool.give_back(self.innerq_cache_release_pages())

    def close(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:
            _lib.innerq_cache_destroy(h)

    def __del__(self):
        try:
            self.close()
        except Exception:       # interpreter shutdown: globals may already be gone
            pass

    @property
    def n_tokens(self) -> int:
        return _check(lib().innerq_cache_n_tokens(self._h), "innerq_cache_n_tokens")

    @property
    def units(self) -> int:
        return self.cfg.batch * self.cfg.n_kv_heads

    def innerq_quantize_prefill(self, k, v, stream=None):
        c = self.cfg
        n = int(k.shape[2]) if k.dim() == 4 else -1
        shape = (c.batch, c.n_kv_heads, n, c.head_dim)
        kp, vp = (_dev_ptr(k, "k", shape, self.device), _dev_ptr(v, "v", shape, self.device)) if n > 0 else (k.data_ptr(), v.data_ptr())
        _check(lib().innerq_quantize_prefill(self._h, kp, vp, n, _stream_ptr(stream, self.device)), "innerq_quantize_prefill")

    def innerq_append_token(self, k_new, v_new, stream=None):
        c = self.cfg
        shape = (c.batch, c.n_kv_heads, c.head_dim)
        _check(lib().innerq_append_token(self._h, _dev_ptr(k_new, "k_new", shape, self.device), _dev_ptr(v_new, "v_new", shape, self.device),
                                         _stream_ptr(stream, self.device)), "innerq_append_token")

    def innerq_decode_attention(self, q, out=None, stream=None):
        import torch
        c = self.cfg
        shape = (c.batch, c.n_q_heads, c.head_dim)
        if out is None:
            out = torch.empty(shape, dtype=torch.float16, device=self.device)
        _check(lib().innerq_decode_attention(self._h, _dev_ptr(q, "q", shape, self.device), _dev_ptr(out, "out", shape, self.device),
                                             _stream_ptr(stream, self.device)), "innerq_decode_attention")
        return out

    # The two calls of a decode step with addresses instead of tensors, for loops that have validated their buffers
    # once (contiguous fp16 CUDA tensors of the shapes above, on this cache's device, which is current) and then
    # step through them by pointer arithmetic: the same C entry points, without the per-call checks.
    def innerq_append_token_ptr(self, k_new_ptr: int, v_new_ptr: int, stream_ptr: int):
        st = _lib.innerq_append_token(self._h, k_new_ptr, v_new_ptr, stream_ptr)
        if st:
            _check(st, "innerq_append_token")

    def innerq_decode_attention_ptr(self, q_ptr: int, out_ptr: int, stream_ptr: int):
        st = _lib.innerq_decode_attention(self._h, q_ptr, out_ptr, stream_ptr)
        if st:
            _check(st, "innerq_decode_attention")

    def innerq_decode_attention_static(self, q, out=None, stream=None):
        """Decode on the library's built-in scratch array: for callers that cannot supply device scratch
        themselves.  Allocates nothing inside the library (the `out` tensor, if not passed, is still a
        normal torch allocation made here in the binding)."""
        import torch
        c = self.cfg
        shape = (c.batch, c.n_q_heads, c.head_dim)
        if out is None:
            out = torch.empty(shape, dtype=torch.float16, device=self.device)
        _check(lib().innerq_decode_attention_static(self._h, _dev_ptr(q, "q", shape, self.device), _dev_ptr(out, "out", shape, self.device),
                                                    _stream_ptr(stream, self.device)), "innerq_decode_attention_static")
        return out

    def innerq_decode_attention_multi(self, q, out=None, stream=None):
        """q fp16 [batch, n_q, n_q_heads, head_dim] (the n_q newest cache tokens are the queries' own) -> out of the
        same shape, causal.  The device scratch the C call needs is a torch allocation made here on first use."""
        import torch
        c = self.cfg
        if not (isinstance(q, torch.Tensor) and q.dim() == 4):
            raise TypeError("q must be a [batch, n_q, n_q_heads, head_dim] tensor")
        n_q = int(q.shape[1])
        shape = (c.batch, n_q, c.n_q_heads, c.head_dim)
        if out is None:
            out = torch.empty(shape, dtype=torch.float16, device=self.device)
        if getattr(self, "_multi_scratch", None) is None:
            n = C.c_size_t()
            _check(lib().innerq_multi_query_scratch_bytes(C.byref(c), C.byref(n)), "innerq_multi_query_scratch_bytes")
            self._multi_scratch = torch.empty(n.value, dtype=torch.uint8, device=self.device)
        _check(lib().innerq_decode_attention_multi(self._h, _dev_ptr(q, "q", shape, self.device), _dev_ptr(out, "out", shape, self.device), n_q,
                                                   self._multi_scratch.data_ptr(), self._multi_scratch.numel(),
                                                   _stream_ptr(stream, self.device)), "innerq_decode_attention_multi")
        return out

    def innerq_decode_step_host(self, k_new_host, v_new_host, q_host, out_host, stream=None):
        """One step (append + decode) from pinned host tensors into a pinned host tensor; enqueues only, the
        caller synchronises the stream before reading `out_host`.  The device staging buffer the C call needs
        is a torch allocation made here on first use."""
        import torch
        c = self.cfg
        kv_shape, q_shape = (c.batch, c.n_kv_heads, c.head_dim), (c.batch, c.n_q_heads, c.head_dim)
        for t, name, shape in ((k_new_host, "k_new_host", kv_shape), (v_new_host, "v_new_host", kv_shape),
                               (q_host, "q_host", q_shape), (out_host, "out_host", q_shape)):
            if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == torch.float16 and t.is_contiguous()
                    and tuple(t.shape) == shape):
                raise TypeError(f"{name} must be a contiguous host fp16 tensor of shape {shape}")
        if getattr(self, "_staging", None) is None:
            n = C.c_size_t()
            _check(lib().innerq_step_staging_bytes(C.byref(c), C.byref(n)), "innerq_step_staging_bytes")
            self._staging = torch.empty(n.value, dtype=torch.uint8, device=self.device)
        _check(lib().innerq_decode_step_host(self._h, k_new_host.data_ptr(), v_new_host.data_ptr(), q_host.data_ptr(),
                                             out_host.data_ptr(), self._staging.data_ptr(), _stream_ptr(stream, self.device)),
               "innerq_decode_step_host")

    def innerq_set_decode_options(self, n_splits: int = 0, variant: int = 0):
        _check(lib().innerq_set_decode_options(self._h, n_splits, variant), "innerq_set_decode_options")

    def innerq_read_device_error(self, stream=None) -> int:
        return _check(lib().innerq_read_device_error(self._h, _stream_ptr(stream, self.device)), "innerq_read_device_error")

    def innerq_selftest_wait_expiry(self, stream=None):
        _check(lib().innerq_selftest_wait_expiry(self._h, _stream_ptr(stream, self.device)), "innerq_selftest_wait_expiry")

    def innerq_last_launch_count(self, which: int) -> int:
        return _check(lib().innerq_last_launch_count(self._h, which), "innerq_last_launch_count")

    def innerq_cache_import(self, arrays: dict, stream=None):
        """Fills the cache from the dict innerq_cache_export returned for a cache of the same configuration (numpy
        arrays trimmed to the live counts; they are padded back to the capacity shapes here and copied to the device)."""
        import torch
        c = self.cfg
        U, D, G, cap = self.units, c.head_dim, c.group, c.max_tokens
        fp16 = c.grouping == GROUPING_FP16
        inner = c.grouping == GROUPING_INNER
        n_tokens = int(arrays["n_tokens"])

        def pad(a, shape, dtype):
            t = torch.zeros(shape, dtype=dtype, device=self.device)
            if a is not None and a.size:
                src = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
                t[tuple(slice(0, n) for n in src.shape)] = src.to(self.device)
            return t

        row_meta, blk_meta = (U, cap, D // G), (U, cap // G + 1, D)
        t = {"norm": pad(arrays["norm"].reshape(U, D), (U, D), torch.float32)}
        sink_cap = cap if fp16 else c.w_sink
        for k in ("k_sink", "v_sink"):
            t[k] = pad(arrays[k], (U, max(sink_cap, 1), D), torch.float16)
        if not fp16:
            km, vm = (row_meta, blk_meta) if inner else (blk_meta, row_meta)
            t["k_code"], t["v_code"] = pad(arrays["k_code"], (U, cap, D), torch.uint8), pad(arrays["v_code"], (U, cap, D), torch.uint8)
            t["k_scale"], t["k_zero"] = pad(arrays["k_scale"], km, torch.int16), pad(arrays["k_zero"], km, torch.int16)
            t["v_scale"], t["v_zero"] = pad(arrays["v_scale"], vm, torch.int16), pad(arrays["v_zero"], vm, torch.int16)
            t["k_recent"] = pad(arrays["k_recent"], (U, c.w_recent + G, D), torch.float16)
            t["v_recent"] = pad(arrays["v_recent"], (U, c.w_recent + G, D), torch.float16)
        ex = innerq_export_t()
        for name, ten in t.items():
            setattr(ex, name, ten.data_ptr())
        _check(lib().innerq_cache_import(self._h, C.byref(ex), n_tokens, _stream_ptr(stream, self.device)), "innerq_cache_import")
        torch.cuda.synchronize(self.device)      # the temporaries above may go once the kernels have read them

    def innerq_cache_export(self, stream=None, codes: bool = True) -> dict:
        """Canonical (unpacked) cache contents as numpy arrays trimmed to the live counts."""
        import torch
        c = self.cfg
        U, D, G, cap = self.units, c.head_dim, c.group, c.max_tokens
        fp16 = c.grouping == GROUPING_FP16
        inner = c.grouping == GROUPING_INNER
        dev = self.device

        def buf(shape, dtype):
            return torch.zeros(shape, dtype=dtype, device=dev)

        row_meta, blk_meta = (U, cap, D // G), (U, cap // G + 1, D)
        t = {}
        if not fp16:
            if codes:
                t["k_code"], t["v_code"] = buf((U, cap, D), torch.uint8), buf((U, cap, D), torch.uint8)
            km, vm = (row_meta, blk_meta) if inner else (blk_meta, row_meta)
            t["k_scale"], t["k_zero"] = buf(km, torch.int16), buf(km, torch.int16)
            t["v_scale"], t["v_zero"] = buf(vm, torch.int16), buf(vm, torch.int16)
            t["k_recent"] = buf((U, c.w_recent + G, D), torch.float16)
            t["v_recent"] = buf((U, c.w_recent + G, D), torch.float16)
        t["norm"] = buf((U, D), torch.float32)
        sink_cap = cap if fp16 else c.w_sink
        t["k_sink"], t["v_sink"] = buf((U, max(sink_cap, 1), D), torch.float16), buf((U, max(sink_cap, 1), D), torch.float16)
        ex = innerq_export_t()
        for name, ten in t.items():
            setattr(ex, name, ten.data_ptr())
        _check(lib().innerq_cache_export(self._h, C.byref(ex), _stream_ptr(stream, self.device)), "innerq_cache_export")
        torch.cuda.synchronize(dev)
        out = {k: getattr(ex, k) for k in ("n_tokens", "n_sink", "n_qk", "n_qv", "n_k_recent", "n_v_recent")}
        host = {k: v.cpu().numpy() for k, v in t.items()}
        out["norm"] = host["norm"]
        out["k_sink"], out["v_sink"] = host["k_sink"][:, :out["n_sink"]], host["v_sink"][:, :out["n_sink"]]
        if fp16:
            return out
        out["k_recent"] = host["k_recent"][:, :out["n_k_recent"]]
        out["v_recent"] = host["v_recent"][:, :out["n_v_recent"]]
        nk_meta = out["n_qk"] if inner else out["n_qk"] // G
        nv_meta = out["n_qv"] // G if inner else out["n_qv"]
        if codes:
            out["k_code"], out["v_code"] = host["k_code"][:, :out["n_qk"]], host["v_code"][:, :out["n_qv"]]
        out["k_scale"] = host["k_scale"].view(np.uint16)[:, :nk_meta]
        out["k_zero"] = host["k_zero"].view(np.uint16)[:, :nk_meta]
        out["v_scale"] = host["v_scale"].view(np.uint16)[:, :nv_meta]
        out["v_zero"] = host["v_zero"].view(np.uint16)[:, :nv_meta]
        return out
