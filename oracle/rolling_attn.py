"""CPU oracle for rolling-KV chunk attention.  TEST INFRASTRUCTURE ONLY.

Plain, slow, fp64 numpy restatement of what the streaming scheme of the paper
computes for one DiT layer (Sec. 3.2 "Rolling KV Cache with Frame Sinks",
Sec. 3.2 "Clip-level Group-wise Sampling", Sec. 3.3 "Streaming Long Tuning").
Nothing here is blocked, fused or reordered, and nothing is shared with the
CUDA path: the product never imports this package, and this package never
imports the product.  Only tests, the smoke check and the CPU-baseline leg of
the benchmark may call it.

The method is exact attention over a restricted key set, so every function is
the plain definition written out.  Inputs are the bf16-rounded values widened
to fp64; all arithmetic is fp64.

Parity pins (tests/test_oracle_pins.py): single key returns its V, identical
keys return the mean of V, softmax rows sum to one, key permutation
invariance, split-merge identity, backward vs central finite differences,
sum-of-dV identity, textbook library attention on the no-eviction special
case, ring cache vs from-scratch masked attention over the whole history.
"""
from __future__ import annotations

from collections import deque

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


class RollingKVCache:
    """Sink + sliding-window cache model (Sec. 3.2, restricted context C_n).

    The first ``sink_frames`` frames ever appended are kept for good; later
    frames enter a window of at most ``window_frames`` frames from which only
    the oldest can be dropped.  Frames are stored as given (bit patterns or
    floats), shape [B_c, T, H, D] each.  There is no implicit eviction.
    """

    def __init__(self, sink_frames: int, window_frames: int):
        self.S = int(sink_frames)
        self.L = int(window_frames)
        self.sink_k: list = []
        self.sink_v: list = []
        self.win_k: deque = deque()
        self.win_v: deque = deque()
        self.frames_seen = 0

    def held(self) -> int:
        return len(self.sink_k) + len(self.win_k)

    def append(self, k_frames: np.ndarray, v_frames: np.ndarray, tokens_per_frame: int) -> None:
        """k_frames, v_frames: [B_c, f*T, H, D]; split into f frames and push in order."""
        T = int(tokens_per_frame)
        assert k_frames.shape == v_frames.shape and k_frames.shape[1] % T == 0
        f = k_frames.shape[1] // T
        room = (self.S - len(self.sink_k)) + (self.L - len(self.win_k))
        if f > room:
            raise OverflowError("append exceeds S+L held frames")
        for j in range(f):
            kf = k_frames[:, j * T:(j + 1) * T].copy()
            vf = v_frames[:, j * T:(j + 1) * T].copy()
            if len(self.sink_k) < self.S:
                self.sink_k.append(kf)
                self.sink_v.append(vf)
            else:
                self.win_k.append(kf)
                self.win_v.append(vf)
            self.frames_seen += 1

    def evict(self, n_frames: int) -> None:
        """Drop the n oldest window frames; sink frames are never dropped."""
        if n_frames > len(self.win_k):
            raise IndexError("evict asks for more window frames than held")
        for _ in range(int(n_frames)):
            self.win_k.popleft()
            self.win_v.popleft()

    def reset(self) -> None:
        self.sink_k.clear(); self.sink_v.clear(); self.win_k.clear(); self.win_v.clear()
        self.frames_seen = 0

    def export(self):
        """Logical contents [B_c, held*T, H, D]: sink frames, then window old -> new."""
        ks = list(self.sink_k) + list(self.win_k)
        vs = list(self.sink_v) + list(self.win_v)
        if not ks:
            return None, None
        return np.concatenate(ks, axis=1), np.concatenate(vs, axis=1)


def _keys_for(b: int, k_ctx, k_c):
    """All keys seen by the chunk queries of sample b: cached context then the chunk itself."""
    parts = []
    if k_ctx is not None and k_ctx.shape[1] > 0:
        parts.append(k_ctx[b if k_ctx.shape[0] > 1 else 0])
    if k_c is not None and k_c.shape[1] > 0:
        parts.append(k_c[b])
    if not parts:
        raise ValueError("empty key set: softmax undefined")
    return np.concatenate(parts, axis=0)  # [N_k, H, D]


def chunk_attn_fwd(q, k_ctx, v_ctx, k_c, v_c, scale: float):
    """Forward of chunk attention against the restricted context (Sec. 3.2).

    q [B, M, H, D]; k_ctx, v_ctx [B_c, N_ctx, H, D] with B_c in {1, B} (B_c = 1
    is the shared frozen prefix of group-wise sampling) or None; k_c, v_c
    [B, n_kc, H, D].  Every query sees every cached key and every chunk key.
    Returns O [B, M, H, D] and LSE [B, H, M] (natural log of sum_j exp(s_ij)).
    """
    q = np.asarray(q, dtype=np.float64)
    B, M, H, D = q.shape
    o = np.zeros((B, M, H, D), dtype=np.float64)
    lse = np.zeros((B, H, M), dtype=np.float64)
    for b in range(B):
        k_all = np.asarray(_keys_for(b, k_ctx, k_c), dtype=np.float64)
        v_all = np.asarray(_keys_for(b, v_ctx, v_c), dtype=np.float64)
        for h in range(H):
            s = scale * (q[b, :, h, :] @ k_all[:, h, :].T)          # s_ij
            m = s.max(axis=1, keepdims=True)                          # m_i
            e = np.exp(s - m)
            z = e.sum(axis=1, keepdims=True)
            lse[b, h, :] = (m + np.log(z))[:, 0]
            p = e / z                                                 # p_ij
            o[b, :, h, :] = p @ v_all[:, h, :]
    return o, lse


def chunk_attn_bwd(q, k_ctx, v_ctx, k_c, v_c, d_o, scale: float, return_full: bool = False):
    """Backward with the cached context detached (Sec. 3.3 "Streaming Long Tuning").

    Given dO, returns dQ (over all keys) and dK, dV of the chunk's own keys only;
    cached keys and values are constants of the graph.  With ``return_full`` the
    gradients of every key (context included) are also returned, for the pins.
    """
    q = np.asarray(q, dtype=np.float64)
    d_o = np.asarray(d_o, dtype=np.float64)
    B, M, H, D = q.shape
    n_kc = 0 if k_c is None else k_c.shape[1]
    dq = np.zeros_like(q)
    dk_c = np.zeros((B, n_kc, H, D), dtype=np.float64)
    dv_c = np.zeros((B, n_kc, H, D), dtype=np.float64)
    full = []
    for b in range(B):
        k_all = np.asarray(_keys_for(b, k_ctx, k_c), dtype=np.float64)
        v_all = np.asarray(_keys_for(b, v_ctx, v_c), dtype=np.float64)
        n_k = k_all.shape[0]
        dk_full = np.zeros((n_k, H, D)); dv_full = np.zeros((n_k, H, D))
        for h in range(H):
            qh, kh, vh, doh = q[b, :, h, :], k_all[:, h, :], v_all[:, h, :], d_o[b, :, h, :]
            s = scale * (qh @ kh.T)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            p = e / e.sum(axis=1, keepdims=True)
            dv = p.T @ doh                                   # dv_j = sum_i p_ij dO_i
            dp = doh @ vh.T                                  # dp_ij = dO_i . v_j
            delta = (p * dp).sum(axis=1, keepdims=True)      # delta_i
            ds = p * (dp - delta)                            # ds_ij
            dq[b, :, h, :] = scale * (ds @ kh)               # all keys
            dk = scale * (ds.T @ qh)
            dk_full[:, h, :] = dk
            dv_full[:, h, :] = dv
        if n_kc:
            dk_c[b] = dk_full[n_k - n_kc:]                   # chunk keys come last in _keys_for
            dv_c[b] = dv_full[n_k - n_kc:]
        full.append((dk_full, dv_full))
    if return_full:
        return dq, dk_c, dv_c, full
    return dq, dk_c, dv_c


def bwd_delta(o, d_o):
    """delta_i = sum_d dO_id * O_id, laid out [B, H, M] (equals sum_j p_ij dp_ij)."""
    o = np.asarray(o, dtype=np.float64); d_o = np.asarray(d_o, dtype=np.float64)
    return np.transpose((o * d_o).sum(axis=-1), (0, 2, 1))


def visibility_mask(n_frames_total: int, chunk_first: int, chunk_frames: int,
                    sink_frames: int, window_frames_held: int) -> np.ndarray:
    """Frame-level visibility of one chunk over the whole streamed history.

    Frame f (index in generation order) is visible to the chunk made of frames
    [chunk_first, chunk_first + chunk_frames) iff it is one of the first
    ``sink_frames`` frames, or one of the ``window_frames_held`` most recent
    frames before the chunk, or a frame of the chunk itself.
    """
    vis = np.zeros(n_frames_total, dtype=bool)
    for f in range(n_frames_total):
        if f >= chunk_first + chunk_frames:
            continue
        if f >= chunk_first:
            vis[f] = True
        elif f < sink_frames:
            vis[f] = True
        elif f >= chunk_first - window_frames_held:
            vis[f] = True
    return vis


def dense_masked_attention(q, k_hist, v_hist, key_visible, scale: float):
    """From-scratch masked attention with no cache model at all.

    q [B, M, H, D]; k_hist, v_hist [B, N_hist, H, D] = every token ever produced;
    key_visible [N_hist] booleans.  Scores of invisible keys are set to -inf.
    Returns O and LSE like ``chunk_attn_fwd``.
    """
    q = np.asarray(q, dtype=np.float64)
    B, M, H, D = q.shape
    o = np.zeros((B, M, H, D)); lse = np.zeros((B, H, M))
    for b in range(B):
        for h in range(H):
            s = scale * (q[b, :, h, :] @ np.asarray(k_hist[b, :, h, :], dtype=np.float64).T)
            s = np.where(key_visible[None, :], s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            z = e.sum(axis=1, keepdims=True)
            lse[b, h] = (m + np.log(z))[:, 0]
            o[b, :, h, :] = (e / z) @ np.asarray(v_hist[b, :, h, :], dtype=np.float64)
    return o, lse
