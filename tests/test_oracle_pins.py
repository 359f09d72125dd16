"""Pins for the CPU oracle: closed forms, invariants, brute force, finite differences.

None of these retype the oracle's formula: each checks it against something the
mathematics fixes independently (or against a library routine on a special case).
"""
import numpy as np
import pytest

from oracle import rolling_attn as orc
from paper_2603_17051_b200 import synth


def rnd(seed, shape):
    return orc.bf16_bits_to_f64(synth.normal_bf16(seed, shape))


def test_bf16_widening_is_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x0000, 0x3DCD, 0x7F80], dtype=np.uint16)
    vals = orc.bf16_bits_to_f64(bits)
    assert vals[0] == 1.0 and vals[1] == -1.0 and vals[2] == 2.0 and vals[3] == 0.0
    assert vals[4] == 0.10009765625 and np.isinf(vals[5])


def test_bf16_rounding_ties_to_even():
    # 1 + 2^-8 is a tie between 1.0 and 1+2^-7: goes to even (1.0); 1 + 3*2^-8 ties up to 1+2^-6
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    v = orc.bf16_bits_to_f64(synth.f32_to_bf16_bits(x))
    assert v[0] == 1.0 and v[1] == 1.0 + 2.0 ** -6 and v[2] == 1.0 + 2.0 ** -7


def test_single_key_returns_its_value():
    q = rnd(1, (2, 5, 3, 8)); k = rnd(2, (2, 1, 3, 8)); v = rnd(3, (2, 1, 3, 8)); do = rnd(4, (2, 5, 3, 8))
    scale = 0.37
    o, lse = orc.chunk_attn_fwd(q, None, None, k, v, scale)
    for i in range(5):
        assert np.array_equal(o[:, i], v[:, 0])
    expect_lse = scale * np.einsum("bihd,bhd->bhi", q, k[:, 0])
    assert np.allclose(lse, expect_lse, atol=1e-13)
    dq, dk, dv = orc.chunk_attn_bwd(q, None, None, k, v, do, scale)
    assert np.abs(dq).max() < 1e-13 and np.abs(dk).max() < 1e-13
    assert np.allclose(dv[:, 0], do.sum(axis=1), atol=1e-12)


def test_identical_keys_give_mean_of_values():
    B, M, H, D, N = 1, 4, 2, 8, 7
    q = rnd(5, (B, M, H, D)); k1 = rnd(6, (B, 1, H, D)); v = rnd(7, (B, N, H, D))
    k = np.repeat(k1, N, axis=1)
    o, lse = orc.chunk_attn_fwd(q, k[:, :3], v[:, :3], k[:, 3:], v[:, 3:], 0.5)
    assert np.allclose(o, np.broadcast_to(v.mean(axis=1, keepdims=True), o.shape), atol=1e-13)
    s = 0.5 * np.einsum("bihd,bhd->bhi", q, k1[:, 0])
    assert np.allclose(lse, s + np.log(N), atol=1e-13)
    # zero queries: uniform weights whatever the keys are
    o0, lse0 = orc.chunk_attn_fwd(np.zeros_like(q), None, None, rnd(8, (B, N, H, D)), v, 0.5)
    assert np.allclose(o0, np.broadcast_to(v.mean(axis=1, keepdims=True), o0.shape), atol=1e-13)
    assert np.allclose(lse0, np.log(N), atol=1e-13)


def test_permutation_of_keys_leaves_o_lse_dq_unchanged():
    B, M, H, D = 2, 6, 2, 16
    q = rnd(10, (B, M, H, D)); kc = rnd(11, (B, 5, H, D)); vc = rnd(12, (B, 5, H, D))
    kx = rnd(13, (B, 9, H, D)); vx = rnd(14, (B, 9, H, D)); do = rnd(15, (B, M, H, D))
    perm = np.random.default_rng(0).permutation(9)
    o1, l1 = orc.chunk_attn_fwd(q, kx, vx, kc, vc, 0.25)
    o2, l2 = orc.chunk_attn_fwd(q, kx[:, perm], vx[:, perm], kc, vc, 0.25)
    assert np.allclose(o1, o2, atol=1e-12) and np.allclose(l1, l2, atol=1e-12)
    g1 = orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, 0.25)
    g2 = orc.chunk_attn_bwd(q, kx[:, perm], vx[:, perm], kc, vc, do, 0.25)
    for a, b in zip(g1, g2):
        assert np.allclose(a, b, atol=1e-12)


def test_split_merge_identity():
    B, M, H, D = 1, 5, 2, 8
    q = rnd(20, (B, M, H, D)); ka = rnd(21, (B, 4, H, D)); va = rnd(22, (B, 4, H, D))
    kb = rnd(23, (B, 6, H, D)); vb = rnd(24, (B, 6, H, D))
    o, lse = orc.chunk_attn_fwd(q, ka, va, kb, vb, 0.3)
    oa, la = orc.chunk_attn_fwd(q, None, None, ka, va, 0.3)
    ob, lb = orc.chunk_attn_fwd(q, None, None, kb, vb, 0.3)
    lm = np.logaddexp(la, lb)
    wa = np.exp(la - lm).transpose(0, 2, 1)[..., None]
    wb = np.exp(lb - lm).transpose(0, 2, 1)[..., None]
    assert np.allclose(lse, lm, atol=1e-12)
    assert np.allclose(o, wa * oa + wb * ob, atol=1e-12)


def test_brute_force_loops_tiny():
    # scalar triple loop straight from the definition, on a tiny case
    B, M, H, D, Nx, Nc = 1, 3, 1, 4, 2, 3
    q = rnd(30, (B, M, H, D)); kx = rnd(31, (B, Nx, H, D)); vx = rnd(32, (B, Nx, H, D))
    kc = rnd(33, (B, Nc, H, D)); vc = rnd(34, (B, Nc, H, D)); scale = 0.5
    o, lse = orc.chunk_attn_fwd(q, kx, vx, kc, vc, scale)
    keys = [kx[0, j, 0] for j in range(Nx)] + [kc[0, j, 0] for j in range(Nc)]
    vals = [vx[0, j, 0] for j in range(Nx)] + [vc[0, j, 0] for j in range(Nc)]
    import math
    for i in range(M):
        s = [scale * sum(q[0, i, 0, d] * kj[d] for d in range(D)) for kj in keys]
        z = sum(math.exp(x) for x in s)
        assert abs(lse[0, 0, i] - math.log(z)) < 1e-12
        for d in range(D):
            ref = sum(math.exp(s[j]) / z * vals[j][d] for j in range(len(keys)))
            assert abs(o[0, i, 0, d] - ref) < 1e-12


def test_rows_sum_to_one_and_dv_total():
    # sum_j dv_j = sum_i dO_i is equivalent to every softmax row summing to one;
    # sum_j ds_ij = 0 per row shows as: dQ is unchanged when a constant vector is added to every key.
    B, M, H, D = 1, 7, 2, 8
    q = rnd(40, (B, M, H, D)); kx = rnd(41, (B, 5, H, D)); vx = rnd(42, (B, 5, H, D))
    kc = rnd(43, (B, 4, H, D)); vc = rnd(44, (B, 4, H, D)); do = rnd(45, (B, M, H, D))
    dq, dk, dv, full = orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, 0.4, return_full=True)
    dv_all = full[0][1]
    assert np.allclose(dv_all.sum(axis=0), do[0].sum(axis=0), atol=1e-12)
    shift = rnd(46, (1, 1, H, D))
    dq2, _, _ = orc.chunk_attn_bwd(q, kx + shift, vx, kc + shift, vc, do, 0.4)
    # p is shift-invariant only per row up to the common factor, so ds is unchanged and dq gains sum_j ds_ij * shift = 0
    assert np.allclose(dq, dq2, atol=1e-11)
    # constant V: O equals that constant (rows sum to one)
    vconst = np.ones_like(vx) * 3.0
    o, _ = orc.chunk_attn_fwd(q, kx, vconst, kc, np.ones_like(vc) * 3.0, 0.4)
    assert np.allclose(o, 3.0, atol=1e-12)


def _loss(q, kx, vx, kc, vc, do, scale):
    o, _ = orc.chunk_attn_fwd(q, kx, vx, kc, vc, scale)
    return float((o * do).sum())


def test_backward_matches_central_finite_differences():
    B, M, H, D = 2, 4, 2, 4
    scale = 0.5
    q = rnd(50, (B, M, H, D)); kx = rnd(51, (B, 3, H, D)); vx = rnd(52, (B, 3, H, D))
    kc = rnd(53, (B, 4, H, D)); vc = rnd(54, (B, 4, H, D)); do = rnd(55, (B, M, H, D))
    dq, dk, dv = orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, scale)
    h = 1e-5
    for name, arr, grad in (("q", q, dq), ("kc", kc, dk), ("vc", vc, dv)):
        num = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = arr[idx]
            arr[idx] = old + h; lp = _loss(q, kx, vx, kc, vc, do, scale)
            arr[idx] = old - h; lm = _loss(q, kx, vx, kc, vc, do, scale)
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        assert np.allclose(num, grad, atol=2e-8), name
    # the context gradient exists mathematically (perturbing a cached key moves the loss) ...
    old = kx[0, 1, 0, 2]
    kx[0, 1, 0, 2] = old + 1e-3; lp = _loss(q, kx, vx, kc, vc, do, scale)
    kx[0, 1, 0, 2] = old - 1e-3; lm = _loss(q, kx, vx, kc, vc, do, scale)
    kx[0, 1, 0, 2] = old
    assert abs(lp - lm) > 1e-7
    # ... and equals the full gradient the oracle computes internally but does not return by default
    _, _, _, full = orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, scale, return_full=True)
    assert abs((lp - lm) / 2e-3 - full[0][0][1, 0, 2]) < 1e-6


def test_shared_prefix_equals_per_sample_copies():
    B, M, H, D = 3, 5, 2, 8
    q = rnd(60, (B, M, H, D)); kx = rnd(61, (1, 6, H, D)); vx = rnd(62, (1, 6, H, D))
    kc = rnd(63, (B, 4, H, D)); vc = rnd(64, (B, 4, H, D)); do = rnd(65, (B, M, H, D))
    o1, l1 = orc.chunk_attn_fwd(q, kx, vx, kc, vc, 0.3)
    o2, l2 = orc.chunk_attn_fwd(q, np.repeat(kx, B, 0), np.repeat(vx, B, 0), kc, vc, 0.3)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)
    g1 = orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, 0.3)
    g2 = orc.chunk_attn_bwd(q, np.repeat(kx, B, 0), np.repeat(vx, B, 0), kc, vc, do, 0.3)
    for a, b in zip(g1, g2):
        assert np.array_equal(a, b)


def test_delta_equals_sum_p_dp():
    B, M, H, D = 1, 5, 2, 8
    q = rnd(70, (B, M, H, D)); kc = rnd(71, (B, 9, H, D)); vc = rnd(72, (B, 9, H, D)); do = rnd(73, (B, M, H, D))
    o, _ = orc.chunk_attn_fwd(q, None, None, kc, vc, 0.35)
    delta = orc.bwd_delta(o, do)
    for h in range(H):
        s = 0.35 * q[0, :, h] @ kc[0, :, h].T
        p = np.exp(s) / np.exp(s).sum(1, keepdims=True)
        dp = do[0, :, h] @ vc[0, :, h].T
        assert np.allclose(delta[0, h], (p * dp).sum(1), atol=1e-12)


def test_no_eviction_matches_library_attention():
    """S=0, nothing evicted: textbook chunk-causal attention; torch SDPA in fp64 as second opinion."""
    torch = pytest.importorskip("torch")
    B, H, D, T, c, n_chunks = 1, 2, 16, 4, 2, 3
    cache = orc.RollingKVCache(0, 8)
    hist_k, hist_v = [], []
    for n in range(n_chunks):
        q = rnd(100 + n, (B, c * T, H, D)); kc = rnd(110 + n, (B, c * T, H, D)); vc = rnd(120 + n, (B, c * T, H, D))
        kx, vx = cache.export()
        o, lse = orc.chunk_attn_fwd(q, kx, vx, kc, vc, 0.25)
        hist_k.append(kc); hist_v.append(vc)
        k_all = torch.from_numpy(np.concatenate(hist_k, 1)).permute(0, 2, 1, 3)
        v_all = torch.from_numpy(np.concatenate(hist_v, 1)).permute(0, 2, 1, 3)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q).permute(0, 2, 1, 3), k_all, v_all, scale=0.25)
        assert np.allclose(o, ref.permute(0, 2, 1, 3).numpy(), atol=1e-10)
        cache.append(kc, vc, T)
    # and with a boolean mask over a longer history (mask hides the future chunk)
    fut_k = rnd(130, (B, c * T, H, D)); fut_v = rnd(131, (B, c * T, H, D))
    k_all = torch.from_numpy(np.concatenate(hist_k + [fut_k], 1)).permute(0, 2, 1, 3)
    v_all = torch.from_numpy(np.concatenate(hist_v + [fut_v], 1)).permute(0, 2, 1, 3)
    mask = torch.ones(c * T, k_all.shape[2], dtype=torch.bool); mask[:, -c * T:] = False
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).permute(0, 2, 1, 3), k_all, v_all, attn_mask=mask, scale=0.25)
    assert np.allclose(o, ref.permute(0, 2, 1, 3).numpy(), atol=1e-10)


@pytest.mark.parametrize("S,L,c,n_chunks", [(0, 6, 3, 4), (1, 6, 3, 5), (3, 5, 2, 7)])
def test_ring_cache_equals_from_scratch_masked_attention(S, L, c, n_chunks):
    """Streaming with evict/append vs dense masked attention over everything ever generated."""
    B, H, D, T = 1, 2, 8, 4
    cache = orc.RollingKVCache(S, L)
    hist_k = np.zeros((B, 0, H, D)); hist_v = np.zeros((B, 0, H, D))
    for n in range(n_chunks):
        # capacity S+L counts every attended frame, the chunk included: evict down to S+L-c held frames
        over = cache.held() - (S + L - c)
        if over > 0:
            cache.evict(over)
        q = rnd(200 + n, (B, c * T, H, D)); kc = rnd(220 + n, (B, c * T, H, D)); vc = rnd(240 + n, (B, c * T, H, D))
        kx, vx = cache.export()
        o, lse = orc.chunk_attn_fwd(q, kx, vx, kc, vc, 0.3)
        hist_k = np.concatenate([hist_k, kc], 1); hist_v = np.concatenate([hist_v, vc], 1)
        frames_total = (n + 1) * c
        win_held = len(cache.win_k)
        vis_f = orc.visibility_mask(frames_total, n * c, c, S, win_held)
        vis = np.repeat(vis_f, T)
        o2, lse2 = orc.dense_masked_attention(q, hist_k, hist_v, vis, 0.3)
        assert np.allclose(o, o2, atol=1e-12) and np.allclose(lse, lse2, atol=1e-12)
        assert cache.held() <= S + L
        # expected visible-frame count: sinks + window + chunk
        assert vis_f.sum() == min(S, n * c) + win_held + c
        cache.append(kc, vc, T)
        assert cache.held() <= S + L


def test_cache_model_sink_retention_and_window_order():
    S, L, T = 2, 4, 3
    cache = orc.RollingKVCache(S, L)
    frames = [synth.normal_bf16(300 + i, (1, T, 2, 4)) for i in range(40)]
    for i, f in enumerate(frames):
        if cache.held() == S + L:
            cache.evict(1)
        cache.append(f, f, T)
        k, v = cache.export()
        held = min(i + 1, S + L)
        assert k.shape[1] == held * T
        expect = frames[:min(S, i + 1)] + frames[max(S, i + 1 - L):i + 1]
        assert np.array_equal(k, np.concatenate(expect, 1))
    with pytest.raises(OverflowError):
        cache.append(frames[0], frames[0], T)
    with pytest.raises(IndexError):
        cache.evict(L + 1)


def test_tiny_stream_matches_stored_oracle_values():
    """Regression guard: the oracle's results on the tiny streamed workload equal the stored values written by
    tests/golden/make_tiny_expected.py (which calls only the oracle)."""
    import importlib.util
    import os
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_tiny_expected", os.path.join(here, "golden", "make_tiny_expected.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    got = mod.tiny_stream_summaries()
    lines = [l.split() for l in open(os.path.join(here, "golden", "tiny_stream_expected.txt")) if not l.startswith("#")]
    assert len(lines) == len(got) == 20
    for (n, name, s, a, e7, e3), ln in zip(got, lines):
        assert int(ln[0]) == n and ln[1] == name
        for val, txt in zip((s, a, e7, e3), ln[2:]):
            assert abs(val - float(txt)) <= 1e-10 * max(1.0, abs(val)), (n, name)
