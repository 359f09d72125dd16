"""ctypes binding of the C ABI declared in include/astro.h.

Argument marshalling only: every step of the path runs in the CUDA kernels of
libastro.so.  There is no fallback: if the library cannot be built or loaded,
or a call returns an error status, an exception is raised.  torch supplies
device memory and the current stream, nothing else.
"""
from __future__ import annotations

import ctypes as C

from . import build as _build

ASTRO_OK = 0
STATUS_NAMES = {0: "ASTRO_OK", 1: "ASTRO_ERR_NULL", 2: "ASTRO_ERR_SHAPE", 3: "ASTRO_ERR_ALIGN",
                4: "ASTRO_ERR_CAPACITY", 5: "ASTRO_ERR_UNDERFLOW", 6: "ASTRO_ERR_ARCH", 7: "ASTRO_ERR_CUDA",
                8: "ASTRO_ERR_TIMEOUT"}

EXPORTED = ("astro_kvcache_key_segments", "astro_selftest_wait_timeout", "astro_nft_loss", "astro_kvcache_get_state", "astro_kvcache_set_state", "astro_kvcache_storage_bytes", "astro_kvcache_create", "astro_kvcache_destroy", "astro_kvcache_reset",
            "astro_kvcache_append", "astro_kvcache_evict", "astro_kvcache_query", "astro_kvcache_export",
            "astro_chunk_attn_fwd", "astro_chunk_attn_bwd_workspace_bytes", "astro_chunk_attn_bwd",
            "astro_chunk_attn_bwd_delta", "astro_chunk_attn_bwd_dq", "astro_chunk_attn_bwd_dkv",
            "astro_chunk_attn_bwd_static", "astro_debug_forward_mode", "astro_debug_pair_flag",
            "astro_last_device_status", "astro_status_string")


class AstroError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s failed: %s (%s)" % (where, STATUS_NAMES.get(self.status, self.status),
                                                  status_string(self.status)))


class KVCacheDesc(C.Structure):
    _fields_ = [("cache_batch", C.c_int), ("heads", C.c_int), ("head_dim", C.c_int),
                ("tokens_per_frame", C.c_int), ("sink_frames", C.c_int), ("window_frames", C.c_int)]


class KVCacheState(C.Structure):
    _fields_ = [("sink_held", C.c_int), ("window_head", C.c_int), ("window_held", C.c_int),
                ("frames_seen", C.c_int64)]


_lib = None


def lib():
    """Load (building first when stale) the shared library; raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = C.CDLL(path)
    vp, ci, cf, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    L.astro_kvcache_storage_bytes.restype = sz
    L.astro_kvcache_storage_bytes.argtypes = [C.POINTER(KVCacheDesc)]
    L.astro_kvcache_create.restype = ci
    L.astro_kvcache_create.argtypes = [C.POINTER(KVCacheDesc), vp, vp, sz, C.POINTER(vp)]
    L.astro_kvcache_destroy.restype = ci
    L.astro_kvcache_destroy.argtypes = [vp]
    L.astro_kvcache_reset.restype = ci
    L.astro_kvcache_reset.argtypes = [vp]
    L.astro_kvcache_append.restype = ci
    L.astro_kvcache_append.argtypes = [vp, vp, vp, ci, vp]
    L.astro_kvcache_evict.restype = ci
    L.astro_kvcache_evict.argtypes = [vp, ci, vp]
    L.astro_kvcache_query.restype = ci
    L.astro_kvcache_query.argtypes = [vp, C.POINTER(ci), C.POINTER(ci), C.POINTER(C.c_int64)]
    L.astro_kvcache_get_state.restype = ci
    L.astro_kvcache_get_state.argtypes = [vp, C.POINTER(KVCacheState)]
    L.astro_kvcache_set_state.restype = ci
    L.astro_kvcache_set_state.argtypes = [vp, C.POINTER(KVCacheState)]
    L.astro_kvcache_key_segments.restype = ci
    L.astro_kvcache_key_segments.argtypes = [vp, ci, C.POINTER(ci), C.POINTER(ci), C.POINTER(ci), C.POINTER(ci)]
    L.astro_kvcache_export.restype = ci
    L.astro_kvcache_export.argtypes = [vp, vp, vp, vp]
    L.astro_chunk_attn_fwd.restype = ci
    L.astro_chunk_attn_fwd.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    L.astro_chunk_attn_bwd_workspace_bytes.restype = sz
    L.astro_chunk_attn_bwd_workspace_bytes.argtypes = [ci, ci, ci, ci]
    L.astro_chunk_attn_bwd.restype = ci
    L.astro_chunk_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, vp, vp, vp, sz, vp]
    L.astro_chunk_attn_bwd_delta.restype = ci
    L.astro_chunk_attn_bwd_delta.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp]
    L.astro_chunk_attn_bwd_dq.restype = ci
    L.astro_chunk_attn_bwd_dq.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, vp]
    L.astro_chunk_attn_bwd_dkv.restype = ci
    L.astro_chunk_attn_bwd_dkv.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    L.astro_chunk_attn_bwd_static.restype = ci
    L.astro_chunk_attn_bwd_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, vp, vp, vp]
    L.astro_nft_loss.restype = ci
    L.astro_nft_loss.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, C.c_longlong, cf, vp, vp, vp, vp]
    L.astro_debug_forward_mode.restype = ci
    L.astro_debug_forward_mode.argtypes = [ci]
    L.astro_debug_pair_flag.restype = ci
    L.astro_debug_pair_flag.argtypes = [C.POINTER(ci)]
    L.astro_selftest_wait_timeout.restype = ci
    L.astro_selftest_wait_timeout.argtypes = [vp]
    L.astro_last_device_status.restype = ci
    L.astro_last_device_status.argtypes = [C.POINTER(C.c_uint32)]
    L.astro_status_string.restype = C.c_char_p
    L.astro_status_string.argtypes = [ci]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().astro_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != ASTRO_OK:
        raise AstroError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _contiguous(*tensors):
    for t in tensors:
        if t is not None and not t.is_contiguous():
            raise ValueError("tensor arguments must be contiguous")


def _used_on(stream, *tensors):
    """Tensors this wrapper allocated are used by kernels on `stream`: tell torch's caching allocator, so that
    a block dropped by the caller is not handed out again (on the allocating stream) while they still run."""
    if stream is None:
        return
    for t in tensors:
        if t is not None:
            t.record_stream(stream)


def _desc(cache_batch, heads, head_dim, tokens_per_frame, sink_frames, window_frames):
    return KVCacheDesc(int(cache_batch), int(heads), int(head_dim), int(tokens_per_frame), int(sink_frames),
                       int(window_frames))


def astro_kvcache_storage_bytes(cache_batch, heads, head_dim, tokens_per_frame, sink_frames, window_frames) -> int:
    d = _desc(cache_batch, heads, head_dim, tokens_per_frame, sink_frames, window_frames)
    return int(lib().astro_kvcache_storage_bytes(C.byref(d)))


class KVCache:
    """Handle of one layer's rolling cache plus the torch tensors that back its storage."""

    def __init__(self, handle, desc, k_storage, v_storage):
        self.handle = handle
        self.desc = desc
        self.k_storage = k_storage
        self.v_storage = v_storage

    def __del__(self):
        try:
            astro_kvcache_destroy(self)
        except Exception:
            pass


def astro_kvcache_create(cache_batch, heads, head_dim, tokens_per_frame, sink_frames, window_frames,
                         k_storage=None, v_storage=None, device="cuda") -> KVCache:
    """Bind storage (torch uint8/bf16 tensors; allocated here with torch when not given) to a new cache."""
    import torch
    d = _desc(cache_batch, heads, head_dim, tokens_per_frame, sink_frames, window_frames)
    nbytes = int(lib().astro_kvcache_storage_bytes(C.byref(d)))
    if nbytes == 0:
        raise AstroError(2, "astro_kvcache_storage_bytes")
    if k_storage is None:
        k_storage = torch.empty(nbytes, dtype=torch.uint8, device=device)
    if v_storage is None:
        v_storage = torch.empty(nbytes, dtype=torch.uint8, device=device)
    out = C.c_void_p()
    st = lib().astro_kvcache_create(C.byref(d), _ptr(k_storage), _ptr(v_storage),
                                    min(k_storage.numel() * k_storage.element_size(),
                                        v_storage.numel() * v_storage.element_size()), C.byref(out))
    _check(st, "astro_kvcache_create")
    return KVCache(out, d, k_storage, v_storage)


def astro_kvcache_destroy(cache: KVCache) -> None:
    if cache.handle is not None and _lib is not None:
        h, cache.handle = cache.handle, None
        _check(_lib.astro_kvcache_destroy(h), "astro_kvcache_destroy")


def astro_kvcache_reset(cache: KVCache) -> None:
    _check(lib().astro_kvcache_reset(cache.handle), "astro_kvcache_reset")


def astro_kvcache_append(cache: KVCache, k, v, n_frames: int, stream=None) -> None:
    """k, v: bf16 [B_c, n_frames*T, H, D] on the device."""
    _check(lib().astro_kvcache_append(cache.handle, _ptr(k), _ptr(v), int(n_frames), _stream(stream)),
           "astro_kvcache_append")


def astro_kvcache_evict(cache: KVCache, n_frames: int, stream=None) -> None:
    _check(lib().astro_kvcache_evict(cache.handle, int(n_frames), None), "astro_kvcache_evict")


def astro_kvcache_query(cache: KVCache):
    """Returns (sink_held, window_held, frames_seen)."""
    a, b, c = C.c_int(), C.c_int(), C.c_int64()
    _check(lib().astro_kvcache_query(cache.handle, C.byref(a), C.byref(b), C.byref(c)), "astro_kvcache_query")
    return a.value, b.value, c.value


def astro_kvcache_get_state(cache: KVCache) -> KVCacheState:
    st = KVCacheState()
    _check(lib().astro_kvcache_get_state(cache.handle, C.byref(st)), "astro_kvcache_get_state")
    return st


def astro_kvcache_set_state(cache: KVCache, state: KVCacheState) -> None:
    _check(lib().astro_kvcache_set_state(cache.handle, C.byref(state)), "astro_kvcache_set_state")


def astro_kvcache_key_segments(cache, n_kc: int):
    """List of (first_token, token_count, from_chunk) the attention kernels would walk (host only)."""
    n = C.c_int()
    a, b, c = (C.c_int * 3)(), (C.c_int * 3)(), (C.c_int * 3)()
    _check(lib().astro_kvcache_key_segments(None if cache is None else cache.handle, int(n_kc), C.byref(n), a, b, c),
           "astro_kvcache_key_segments")
    return [(a[i], b[i], c[i]) for i in range(n.value)]


def astro_kvcache_export(cache: KVCache, stream=None):
    """Held frames in logical order as two bf16 tensors [B_c, held*T, H, D]."""
    import torch
    sink, win, _ = astro_kvcache_query(cache)
    d = cache.desc
    shape = (d.cache_batch, (sink + win) * d.tokens_per_frame, d.heads, d.head_dim)
    k = torch.empty(shape, dtype=torch.bfloat16, device=cache.k_storage.device)
    v = torch.empty_like(k)
    if sink + win:
        _check(lib().astro_kvcache_export(cache.handle, _ptr(k), _ptr(v), _stream(stream)), "astro_kvcache_export")
    return k, v


def astro_chunk_attn_fwd(cache, q, k_chunk, v_chunk, scale: float, o=None, lse=None, stream=None):
    """q [B, n_q, H, D], k_chunk/v_chunk [B, n_kc, H, D] or None; returns (O bf16, LSE fp32 [B, H, n_q])."""
    import torch
    B, n_q, H, D = q.shape
    n_kc = 0 if k_chunk is None else k_chunk.shape[1]
    fresh = []
    if o is None:
        o = torch.empty_like(q); fresh.append(o)
    if lse is None:
        lse = torch.empty((B, H, n_q), dtype=torch.float32, device=q.device); fresh.append(lse)
    _contiguous(q, k_chunk, v_chunk, o, lse)
    _used_on(stream, *fresh)
    st = lib().astro_chunk_attn_fwd(None if cache is None else cache.handle, _ptr(q), _ptr(k_chunk), _ptr(v_chunk),
                                    B, H, D, n_q, n_kc, float(scale), _ptr(o), _ptr(lse), _stream(stream))
    _check(st, "astro_chunk_attn_fwd")
    return o, lse


def astro_chunk_attn_bwd_workspace_bytes(batch, heads, n_q, head_dim) -> int:
    return int(lib().astro_chunk_attn_bwd_workspace_bytes(int(batch), int(heads), int(n_q), int(head_dim)))


def astro_chunk_attn_bwd(cache, q, k_chunk, v_chunk, o, lse, d_o, scale: float, dq=None, dk_chunk=None,
                         dv_chunk=None, workspace=None, stream=None):
    """Returns (dQ, dK_chunk, dV_chunk), bf16; the cached context receives no gradient."""
    import torch
    B, n_q, H, D = q.shape
    n_kc = 0 if k_chunk is None else k_chunk.shape[1]
    fresh = []
    if dq is None:
        dq = torch.empty_like(q); fresh.append(dq)
    if n_kc and dk_chunk is None:
        dk_chunk = torch.empty_like(k_chunk); fresh.append(dk_chunk)
    if n_kc and dv_chunk is None:
        dv_chunk = torch.empty_like(v_chunk); fresh.append(dv_chunk)
    need = astro_chunk_attn_bwd_workspace_bytes(B, H, n_q, D)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device); fresh.append(workspace)
    _contiguous(q, k_chunk, v_chunk, o, lse, d_o, dq, dk_chunk, dv_chunk)
    _used_on(stream, *fresh)
    st = lib().astro_chunk_attn_bwd(None if cache is None else cache.handle, _ptr(q), _ptr(k_chunk), _ptr(v_chunk),
                                    _ptr(o), _ptr(lse), _ptr(d_o), B, H, D, n_q, n_kc, float(scale), _ptr(dq),
                                    _ptr(dk_chunk), _ptr(dv_chunk), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "astro_chunk_attn_bwd")
    return dq, dk_chunk, dv_chunk


def astro_chunk_attn_bwd_delta(o, d_o, delta=None, stream=None):
    """delta [B, H, n_q] fp32 = rowsum(dO * O)."""
    import torch
    B, n_q, H, D = o.shape
    if delta is None:
        delta = torch.empty((B, H, n_q), dtype=torch.float32, device=o.device)
        _used_on(stream, delta)
    _contiguous(o, d_o, delta)
    _check(lib().astro_chunk_attn_bwd_delta(_ptr(o), _ptr(d_o), B, H, D, n_q, _ptr(delta), _stream(stream)),
           "astro_chunk_attn_bwd_delta")
    return delta


def astro_chunk_attn_bwd_dq(cache, q, k_chunk, v_chunk, lse, delta, d_o, scale: float, dq=None, stream=None):
    import torch
    B, n_q, H, D = q.shape
    n_kc = 0 if k_chunk is None else k_chunk.shape[1]
    if dq is None:
        dq = torch.empty_like(q)
        _used_on(stream, dq)
    _contiguous(q, k_chunk, v_chunk, lse, delta, d_o, dq)
    st = lib().astro_chunk_attn_bwd_dq(None if cache is None else cache.handle, _ptr(q), _ptr(k_chunk), _ptr(v_chunk),
                                       _ptr(lse), _ptr(delta), _ptr(d_o), B, H, D, n_q, n_kc, float(scale), _ptr(dq),
                                       _stream(stream))
    _check(st, "astro_chunk_attn_bwd_dq")
    return dq


def astro_chunk_attn_bwd_dkv(q, k_chunk, v_chunk, lse, delta, d_o, scale: float, dk_chunk=None, dv_chunk=None,
                             stream=None):
    import torch
    B, n_q, H, D = q.shape
    n_kc = k_chunk.shape[1]
    if dk_chunk is None:
        dk_chunk = torch.empty_like(k_chunk)
        _used_on(stream, dk_chunk)
    if dv_chunk is None:
        dv_chunk = torch.empty_like(v_chunk)
        _used_on(stream, dv_chunk)
    _contiguous(q, k_chunk, v_chunk, lse, delta, d_o, dk_chunk, dv_chunk)
    st = lib().astro_chunk_attn_bwd_dkv(_ptr(q), _ptr(k_chunk), _ptr(v_chunk), _ptr(lse), _ptr(delta), _ptr(d_o), B, H,
                                        D, n_q, n_kc, float(scale), _ptr(dk_chunk), _ptr(dv_chunk), _stream(stream))
    _check(st, "astro_chunk_attn_bwd_dkv")
    return dk_chunk, dv_chunk


def astro_nft_loss(v_theta, v_old, v_ref, v_target, r_tilde, beta: float, w_policy=None, w_kl=None, grad=True,
                   stream=None, out=None):
    """Per-sample policy loss and squared distance to the reference, plus d/d v_theta of the weighted total.

    Velocity tensors: bf16 [B, ...] (flattened per sample); r_tilde / weights: fp32 [B].  Returns
    (policy[B], kl[B] or None, grad like v_theta or None); `out` may pass those three preallocated."""
    import torch
    B = v_theta.shape[0]
    elems = v_theta.numel() // B
    if out is not None:
        policy, kl, g = out
    else:
        policy = torch.empty(B, dtype=torch.float32, device=v_theta.device)
        kl = None if v_ref is None else torch.empty(B, dtype=torch.float32, device=v_theta.device)
        g = torch.empty_like(v_theta) if grad else None
        _used_on(stream, policy, kl, g)
    _contiguous(v_theta, v_old, v_ref, v_target, g)
    st = lib().astro_nft_loss(_ptr(v_theta), _ptr(v_old), _ptr(v_ref), _ptr(v_target), _ptr(r_tilde), _ptr(w_policy),
                              _ptr(w_kl), B, elems, float(beta), _ptr(policy), _ptr(kl), _ptr(g), _stream(stream))
    _check(st, "astro_nft_loss")
    return policy, kl, g


BWD_STATIC_MAX_ROWS = 262144


def astro_chunk_attn_bwd_static(cache, q, k_chunk, v_chunk, o, lse, d_o, scale: float, dq, dk_chunk, dv_chunk,
                                stream=None):
    """Backward for callers that may not allocate: no workspace argument, delta goes to a fixed 1 MiB
    device array inside the library (batch * heads * n_q <= BWD_STATIC_MAX_ROWS).  The caller passes every
    output tensor; this wrapper allocates nothing either.  Calls that may overlap on the GPU race on the
    shared array; issue them on one stream."""
    B, n_q, H, D = q.shape
    n_kc = 0 if k_chunk is None else k_chunk.shape[1]
    _contiguous(q, k_chunk, v_chunk, o, lse, d_o, dq, dk_chunk, dv_chunk)
    st = lib().astro_chunk_attn_bwd_static(None if cache is None else cache.handle, _ptr(q), _ptr(k_chunk),
                                           _ptr(v_chunk), _ptr(o), _ptr(lse), _ptr(d_o), B, H, D, n_q, n_kc,
                                           float(scale), _ptr(dq), _ptr(dk_chunk), _ptr(dv_chunk), _stream(stream))
    _check(st, "astro_chunk_attn_bwd_static")
    return dq, dk_chunk, dv_chunk


FWD_MODE_NORMAL, FWD_MODE_SAFE_ONLY, FWD_MODE_PAIR = 0, 1, 2


def astro_debug_forward_mode(mode: int) -> None:
    """Diagnostic switch: 0 normal operation, 1 every later forward runs its safe pass only, 2 head_dim 128
    forwards run the CTA-pair kernel."""
    _check(lib().astro_debug_forward_mode(int(mode)), "astro_debug_forward_mode")


def astro_debug_pair_flag() -> int:
    """Synchronises; 1 if a CTA-pair forward since the last call had a row that needs the safe pass (cleared)."""
    f = C.c_int()
    _check(lib().astro_debug_pair_flag(C.byref(f)), "astro_debug_pair_flag")
    return f.value


def astro_selftest_wait_timeout(stream=None) -> None:
    """Enqueue the bounded-wait self-test kernel (its wait runs out on purpose; see astro_last_device_status)."""
    _check(lib().astro_selftest_wait_timeout(_stream(stream)), "astro_selftest_wait_timeout")


def astro_last_device_status() -> int:
    """Synchronises, reads and clears the device status word; raises AstroError on a recorded timeout."""
    detail = C.c_uint32()
    st = lib().astro_last_device_status(C.byref(detail))
    _check(st, "astro_last_device_status (detail 0x%x)" % detail.value)
    return detail.value
