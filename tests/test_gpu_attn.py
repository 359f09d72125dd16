"""GPU parity of chunk attention forward and backward against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest

from helpers import check_fwd, check_grads, dev_bf16, f64, host_bits, rel_l2
from oracle import rolling_attn as orc
from paper_2603_17051_b200 import synth

pytestmark = pytest.mark.gpu


def _ctx(model):
    mk, mv = model.export()
    if mk is None:
        return None, None
    return orc.bf16_bits_to_f64(mk), orc.bf16_bits_to_f64(mv)


def _fill(A, Bc, H, D, T, S, L, held, seed, churn=0):
    """Cache + model holding `held` frames; `churn` extra evict/append rounds move the ring head."""
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L)
    model = orc.RollingKVCache(S, L)
    if held:
        kb = synth.normal_bf16(seed, (Bc, held * T, H, D)); vb = synth.normal_bf16(seed + 1, (Bc, held * T, H, D))
        A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), held); model.append(kb, vb, T)
    for r in range(churn):
        n = min(2, len(model.win_k))
        if n == 0:
            break
        A.astro_kvcache_evict(cache, n); model.evict(n)
        kb = synth.normal_bf16(seed + 10 + 2 * r, (Bc, n * T, H, D)); vb = synth.normal_bf16(seed + 11 + 2 * r, (Bc, n * T, H, D))
        A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), n); model.append(kb, vb, T)
    return cache, model


@pytest.fixture
def safe_pass_only():
    """Every forward inside the test runs the kernel's safe pass (running row reference) instead of the fast one."""
    from paper_2603_17051_b200 import binding as A
    A.astro_debug_forward_mode(A.FWD_MODE_SAFE_ONLY)
    yield
    A.astro_debug_forward_mode(A.FWD_MODE_NORMAL)


@pytest.fixture
def pair_kernel():
    """head_dim 128 forwards inside the test run the CTA-pair kernel; none of them may ask for the safe pass."""
    from paper_2603_17051_b200 import binding as A
    A.astro_debug_pair_flag()
    A.astro_debug_forward_mode(A.FWD_MODE_PAIR)
    yield
    A.astro_debug_forward_mode(A.FWD_MODE_NORMAL)
    assert A.astro_debug_pair_flag() == 0


def _run_case(A, B, Bc, H, D, T, S, L, held, n_q, n_kc, seed, churn=0, evict_hole=0, scale=None, bwd=True,
              sharp=False):
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    cache, model = _fill(A, Bc, H, D, T, S, L, held, seed, churn)
    if evict_hole:
        A.astro_kvcache_evict(cache, evict_hole); model.evict(evict_hole)
    bits = [synth.normal_bf16(seed + 100 + i, shp) for i, shp in
            enumerate(((B, n_q, H, D), (B, n_kc, H, D), (B, n_kc, H, D), (B, n_q, H, D)))]
    q, kc, vc, do = (dev_bf16(x) for x in bits)
    qf, kf, vf, dof = (orc.bf16_bits_to_f64(x) for x in bits)
    if n_kc == 0:
        kc = vc = None
    kx, vx = _ctx(model)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, scale)
    A.astro_last_device_status()
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, kx, vx, kf, vf, scale)
    check_fwd(o, lse, o_ref, lse_ref, sharp=sharp)
    if bwd:
        g = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, scale)
        A.astro_last_device_status()
        g_ref = orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, scale)
        check_grads(g, g_ref)
    return cache, model


def test_tiny_config_streamed_four_chunks():
    """The tiny workload end to end: 4 chunks with evict/append, forward and backward each chunk, exhaustive."""
    from paper_2603_17051_b200 import binding as A
    w = synth.TINY
    cache = A.astro_kvcache_create(w.cache_batch, w.heads, w.head_dim, w.tokens_per_frame, w.sink_frames, w.window_frames)
    model = orc.RollingKVCache(w.sink_frames, w.window_frames)
    M = w.chunk_tokens
    for n in range(4):
        over = model.held() - (w.sink_frames + w.window_frames - w.chunk_frames)
        if over > 0:
            A.astro_kvcache_evict(cache, over); model.evict(over)
        bits = [synth.normal_bf16(synth.tensor_seed(1, 10 * n + i), (w.batch, M, w.heads, w.head_dim)) for i in range(4)]
        q, kc, vc, do = (dev_bf16(x) for x in bits)
        qf, kf, vf, dof = (orc.bf16_bits_to_f64(x) for x in bits)
        kx, vx = _ctx(model)
        o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale)
        g = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, w.scale)
        A.astro_last_device_status()
        check_fwd(o, lse, *orc.chunk_attn_fwd(qf, kx, vx, kf, vf, w.scale), tag="chunk %d" % n)
        check_grads(g, orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, w.scale), tag="chunk %d" % n)
        A.astro_kvcache_append(cache, kc, vc, w.chunk_frames); model.append(bits[1], bits[2], w.tokens_per_frame)
        ke, ve = A.astro_kvcache_export(cache)
        mk, mv = model.export()
        assert np.array_equal(host_bits(ke), mk) and np.array_equal(host_bits(ve), mv)


PARITY_CASES = [
    # several tiles with ragged tails everywhere, per-sample caches, wrapped ring
    dict(B=2, Bc=2, H=3, D=128, T=100, S=1, L=5, held=6, n_q=300, n_kc=300, seed=100, churn=2),
    # shared frozen prefix (B_c = 1) broadcast over a group of 3
    dict(B=3, Bc=1, H=2, D=128, T=50, S=2, L=6, held=8, n_q=333, n_kc=77, seed=200, churn=3),
    # head_dim 64, a hole left by evict without re-append
    dict(B=1, Bc=1, H=2, D=64, T=33, S=1, L=7, held=8, n_q=130, n_kc=99, seed=300, churn=2, evict_hole=3),
    # no cached context at all; n_q != n_kc
    dict(B=2, Bc=2, H=2, D=128, T=16, S=0, L=2, held=0, n_q=200, n_kc=129, seed=400),
    # context only, no chunk keys
    dict(B=1, Bc=1, H=2, D=64, T=40, S=0, L=5, held=5, n_q=64, n_kc=0, seed=500),
    # one query, one key
    dict(B=1, Bc=1, H=1, D=64, T=1, S=0, L=1, held=0, n_q=1, n_kc=1, seed=600),
    # sink only partly filled
    dict(B=1, Bc=1, H=1, D=128, T=10, S=4, L=3, held=2, n_q=17, n_kc=5, seed=700),
    # exact multiples of the tile
    dict(B=1, Bc=1, H=2, D=128, T=128, S=1, L=3, held=4, n_q=256, n_kc=256, seed=800, churn=1),
    # a scale other than 1/sqrt(D): near one-hot softmax.  O is then about one V row (|v| up to ~4.5), and the
    # rounding of the bf16 output alone (half an ulp, up to 7.8e-3 at |o| >= 4) leaves no room inside a flat
    # 1e-2, so each element is held to 1e-2 + half a bf16 ulp of its reference value (helpers.check_fwd)
    dict(B=1, Bc=1, H=2, D=128, T=64, S=0, L=6, held=6, n_q=200, n_kc=100, seed=900, scale=0.7, sharp=True),
    # head_dim 64 with 3 query tiles and 12 key tiles over three segments (wrapped ring + chunk): the 3-deep
    # K and V rings and the two S buffers wrap several times
    dict(B=2, Bc=2, H=2, D=64, T=96, S=2, L=8, held=10, n_q=300, n_kc=290, seed=950, churn=3),
]


@pytest.mark.parametrize("case", PARITY_CASES)
def test_parity_cases(case):
    from paper_2603_17051_b200 import binding as A
    _run_case(A, **case)


@pytest.mark.parametrize("case", [c for c in PARITY_CASES if c["D"] == 128])
def test_parity_cases_pair_kernel(case, pair_kernel):
    """The head_dim 128 cases through the CTA-pair kernel (two query tiles per K/V tile, cta_group::2 MMAs): odd and
    even numbers of query tiles, ragged key ranges, holes, a shared prefix."""
    from paper_2603_17051_b200 import binding as A
    _run_case(A, bwd=False, **case)


@pytest.mark.parametrize("case", PARITY_CASES)
def test_parity_cases_safe_pass(case, safe_pass_only):
    """The same cases through the forward's safe pass (running row reference, O rescaled on the way)."""
    from paper_2603_17051_b200 import binding as A
    _run_case(A, bwd=False, **case)


def test_single_key_and_identical_keys_closed_forms_on_gpu():
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, n_q = 1, 2, 64, 70
    q = dev_bf16(synth.normal_bf16(1, (B, n_q, H, D)))
    v1 = dev_bf16(synth.normal_bf16(2, (B, 1, H, D))); k1 = dev_bf16(synth.normal_bf16(3, (B, 1, H, D)))
    o, lse = A.astro_chunk_attn_fwd(None, q, k1, v1, 0.125)
    assert torch.equal(o, v1.expand(B, n_q, H, D))                      # one key: O is its V, exactly
    kk = k1.expand(B, 37, H, D).contiguous()
    vv = dev_bf16(synth.normal_bf16(4, (B, 37, H, D)))
    o, lse2 = A.astro_chunk_attn_fwd(None, q, kk, vv, 0.125)
    assert (o.float() - vv.float().mean(1, keepdim=True)).abs().max() < 1e-2
    assert (lse2 - (lse + float(np.log(37)))).abs().max() < 1e-3


def test_shared_prefix_equals_replicated_caches():
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, T, S, L, held = 3, 2, 128, 30, 1, 4, 5
    c1 = A.astro_kvcache_create(1, H, D, T, S, L); cB = A.astro_kvcache_create(B, H, D, T, S, L)
    k = dev_bf16(synth.normal_bf16(11, (1, held * T, H, D))); v = dev_bf16(synth.normal_bf16(12, (1, held * T, H, D)))
    A.astro_kvcache_append(c1, k, v, held)
    A.astro_kvcache_append(cB, k.expand(B, -1, -1, -1).contiguous(), v.expand(B, -1, -1, -1).contiguous(), held)
    q, kc, vc, do = (dev_bf16(synth.normal_bf16(13 + i, (B, 90, H, D))) for i in range(4))
    o1, l1 = A.astro_chunk_attn_fwd(c1, q, kc, vc, 0.1)
    oB, lB = A.astro_chunk_attn_fwd(cB, q, kc, vc, 0.1)
    assert torch.equal(o1, oB) and torch.equal(l1, lB)
    g1 = A.astro_chunk_attn_bwd(c1, q, kc, vc, o1, l1, do, 0.1)
    gB = A.astro_chunk_attn_bwd(cB, q, kc, vc, oB, lB, do, 0.1)
    for a, b in zip(g1, gB):
        assert torch.equal(a, b)


@pytest.mark.parametrize("mode", [0, 2])
def test_stale_nan_in_evicted_slots_does_not_leak(mode):
    """Tile rows past a segment's end may hold anything (here NaN): results must not change."""
    import torch
    from paper_2603_17051_b200 import binding as A
    A.astro_debug_forward_mode(mode)
    try:
        _stale_nan_case(A, torch)
    finally:
        A.astro_debug_forward_mode(0)


def _stale_nan_case(A, torch):
    H, D, T, S, L = 2, 128, 50, 0, 4
    cache = A.astro_kvcache_create(1, H, D, T, S, L)
    cache.k_storage.view(torch.int16).fill_(0x7FC0 - 0x10000 if False else 0x7FC0)
    cache.v_storage.view(torch.int16).fill_(0x7FC0)
    model = orc.RollingKVCache(S, L)
    kb = synth.normal_bf16(21, (1, 3 * T, H, D)); vb = synth.normal_bf16(22, (1, 3 * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), 3); model.append(kb, vb, T)
    bits = [synth.normal_bf16(23 + i, (1, 60, H, D)) for i in range(4)]
    q, kc, vc, do = (dev_bf16(x) for x in bits)
    qf, kf, vf, dof = (orc.bf16_bits_to_f64(x) for x in bits)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, 0.09)
    g = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, 0.09)
    kx, vx = _ctx(model)
    check_fwd(o, lse, *orc.chunk_attn_fwd(qf, kx, vx, kf, vf, 0.09))
    check_grads(g, orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, 0.09))


def test_canary_padding_around_outputs_is_untouched():
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, n_q, n_kc = 1, 2, 128, 150, 140
    pad = 4096
    def padded(shape, dtype):
        n = int(np.prod(shape))
        buf = torch.full((n + 2 * pad,), 7, dtype=dtype, device="cuda")
        return buf, buf[pad:pad + n].view(shape)
    q, kc, vc, do = (dev_bf16(synth.normal_bf16(31 + i, (B, n, H, D))) for i, n in enumerate((n_q, n_kc, n_kc, n_q)))
    ob, o = padded((B, n_q, H, D), torch.bfloat16); lb, lse = padded((B, H, n_q), torch.float32)
    A.astro_chunk_attn_fwd(None, q, kc, vc, 0.1, o=o, lse=lse)
    dqb, dq = padded((B, n_q, H, D), torch.bfloat16); dkb, dk = padded((B, n_kc, H, D), torch.bfloat16)
    dvb, dv = padded((B, n_kc, H, D), torch.bfloat16)
    A.astro_chunk_attn_bwd(None, q, kc, vc, o, lse, do, 0.1, dq=dq, dk_chunk=dk, dv_chunk=dv)
    A.astro_last_device_status()
    for buf in (ob, lb, dqb, dkb, dvb):
        assert (buf[:pad] == 7).all() and (buf[-pad:] == 7).all()


def _sample_rows(n_q, n_rand, rng):
    tail = np.arange((n_q // 128) * 128, n_q)                       # every row of the ragged last tile
    rows = np.unique(np.concatenate([rng.choice(n_q, n_rand, replace=False), tail, [0, 127, 128]]))
    return rows


def test_layer_shape_forward_sampled_rows():
    """Full-size single-layer forward (12 heads, D=128, 4680 queries x 32760 keys) in the launch
    configuration the benchmark times; the oracle computes sampled query rows one by one."""
    from paper_2603_17051_b200 import binding as A
    w = synth.LAYER_FWD
    cache, model = _fill(A, w.cache_batch, w.heads, w.head_dim, w.tokens_per_frame, w.sink_frames,
                         w.window_frames, w.held_frames, synth.tensor_seed(2, 0), churn=2)
    bits = [synth.normal_bf16(synth.tensor_seed(2, 50 + i), (w.batch, w.chunk_tokens, w.heads, w.head_dim)) for i in range(3)]
    q, kc, vc = (dev_bf16(x) for x in bits)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale)
    A.astro_last_device_status()
    rows = _sample_rows(w.chunk_tokens, 64, np.random.default_rng(2))
    kx, vx = _ctx(model)
    qf, kf, vf = (orc.bf16_bits_to_f64(x) for x in bits)
    o_ref, lse_ref = orc.chunk_attn_fwd(qf[:, rows], kx, vx, kf, vf, w.scale)
    check_fwd(o[:, rows], lse[:, :, rows], o_ref, lse_ref)


def test_rl_update_shape_backward_sampled():
    """Full-size clip-window update (batch 2, 28080 detached keys + 4680 trainable): dQ on sampled rows
    (rows are independent), dK/dV in full for two (sample, head) pairs."""
    from paper_2603_17051_b200 import binding as A
    w = synth.RL_UPDATE
    cache, model = _fill(A, w.cache_batch, w.heads, w.head_dim, w.tokens_per_frame, w.sink_frames,
                         w.window_frames, w.held_frames, synth.tensor_seed(4, 0), churn=1)
    bits = [synth.normal_bf16(synth.tensor_seed(4, 50 + i), (w.batch, w.chunk_tokens, w.heads, w.head_dim)) for i in range(4)]
    q, kc, vc, do = (dev_bf16(x) for x in bits)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale)
    dq, dk, dv = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, w.scale)
    A.astro_last_device_status()
    mk, mv = model.export()
    rows = _sample_rows(w.chunk_tokens, 48, np.random.default_rng(4))
    for (b, h) in ((0, 3), (1, 11)):
        sl = lambda x: orc.bf16_bits_to_f64(x[b:b + 1, :, h:h + 1, :])
        qf, kf, vf, dof, kx, vx = sl(bits[0]), sl(bits[1]), sl(bits[2]), sl(bits[3]), sl(mk), sl(mv)
        o_ref, lse_ref = orc.chunk_attn_fwd(qf, kx, vx, kf, vf, w.scale)
        check_fwd(o[b:b + 1, :, h:h + 1], lse[b:b + 1, h:h + 1], o_ref, lse_ref, tag="b%d h%d" % (b, h))
        dq_ref, dk_ref, dv_ref = orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, w.scale)
        check_grads((dq[b:b + 1, :, h:h + 1], dk[b:b + 1, :, h:h + 1], dv[b:b + 1, :, h:h + 1]),
                    (dq_ref, dk_ref, dv_ref), tag="b%d h%d" % (b, h))
        e = rel_l2(f64(dq[b:b + 1, rows, h:h + 1]), dq_ref[:, rows])
        assert e <= 1e-2, "sampled dQ rows rel-L2 %.3e" % e


def test_rollout_shape_streamed_eight_chunks_sampled():
    """Long-rollout shape (batch 4, per-sample caches, 3 sink + 12 window slots, 1560 tokens per frame):
    eight chunks streamed so that the ring wraps; cache bit-exact, forward of the last chunk on sampled rows."""
    from paper_2603_17051_b200 import binding as A
    w = synth.ROLLOUT
    H, D, T, c, M = w.heads, w.head_dim, w.tokens_per_frame, w.chunk_frames, w.chunk_tokens
    cache = A.astro_kvcache_create(w.batch, H, D, T, w.sink_frames, w.window_frames)
    model = orc.RollingKVCache(w.sink_frames, w.window_frames)
    cap = w.sink_frames + w.window_frames
    for n in range(8):
        over = model.held() - (cap - c)
        if over > 0:
            A.astro_kvcache_evict(cache, over); model.evict(over)
        kb = synth.normal_bf16(synth.tensor_seed(3, 2 * n), (w.batch, M, H, D))
        vb = synth.normal_bf16(synth.tensor_seed(3, 2 * n + 1), (w.batch, M, H, D))
        kc, vc = dev_bf16(kb), dev_bf16(vb)
        if n == 7:
            qb = synth.normal_bf16(synth.tensor_seed(3, 100), (w.batch, M, H, D))
            q = dev_bf16(qb)
            for _ in range(4):                                   # four denoising steps against a fixed cache
                o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale)
            A.astro_last_device_status()
            assert model.held() == 12
            mk, mv = model.export()
            rows = _sample_rows(M, 48, np.random.default_rng(3))
            for (b, h) in ((0, 0), (3, 7)):
                sl = lambda x: orc.bf16_bits_to_f64(x[b:b + 1, :, h:h + 1, :])
                o_ref, lse_ref = orc.chunk_attn_fwd(sl(qb)[:, rows], sl(mk), sl(mv), sl(kb), sl(vb), w.scale)
                check_fwd(o[b:b + 1, rows, h:h + 1], lse[b:b + 1, h:h + 1][:, :, rows], o_ref, lse_ref, tag="b%d h%d" % (b, h))
        A.astro_kvcache_append(cache, kc, vc, c); model.append(kb, vb, T)
    ke, ve = A.astro_kvcache_export(cache)
    mk, mv = model.export()
    assert np.array_equal(host_bits(ke), mk) and np.array_equal(host_bits(ve), mv)
    assert A.astro_kvcache_query(cache) == (3, 12, 24)


def test_longest_sweep_context_sampled():
    """65520 keys per query (60840 cached as 78 half-frames of 780 tokens + the 4680-token chunk), batch 2 of the
    sweep's 8 samples: forward on sampled rows."""
    from paper_2603_17051_b200 import binding as A
    B, H, D, T, frames, M = 2, 12, 128, 780, 78, 4680
    cache = A.astro_kvcache_create(B, H, D, T, 0, frames)
    kxb = synth.normal_bf16(synth.tensor_seed(5, 0), (B, frames * T, H, D))
    vxb = synth.normal_bf16(synth.tensor_seed(5, 1), (B, frames * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kxb), dev_bf16(vxb), frames)
    bits = [synth.normal_bf16(synth.tensor_seed(5, 10 + i), (B, M, H, D)) for i in range(3)]
    q, kc, vc = (dev_bf16(x) for x in bits)
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, scale)
    A.astro_last_device_status()
    rows = _sample_rows(M, 48, np.random.default_rng(5))
    for (b, h) in ((0, 5), (1, 11)):
        sl = lambda x: orc.bf16_bits_to_f64(x[b:b + 1, :, h:h + 1, :])
        o_ref, lse_ref = orc.chunk_attn_fwd(sl(bits[0])[:, rows], sl(kxb), sl(vxb), sl(bits[1]), sl(bits[2]), scale)
        check_fwd(o[b:b + 1, rows, h:h + 1], lse[b:b + 1, h:h + 1][:, :, rows], o_ref, lse_ref, tag="b%d h%d" % (b, h))


@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_and_cache_histories(seed):
    """Seeded fuzz: random head counts, frame sizes, sink/window sizes, cache histories (wraps, holes, partly
    filled sinks), query/key counts around tile boundaries, shared or per-sample caches; forward and backward."""
    from paper_2603_17051_b200 import binding as A
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    H = int(rng.integers(1, 4))
    T = int(rng.choice([1, 7, 16, 31, 64, 100, 129]))
    S = int(rng.integers(0, 3))
    L = int(rng.integers(1, 6))
    B = int(rng.integers(1, 4))
    Bc = int(rng.choice([1, B]))
    held = int(rng.integers(0, S + L + 1))
    n_q = int(rng.choice([1, 5, 127, 128, 129, 200, 257]))
    n_kc = int(rng.choice([0, 1, 63, 64, 65, 128, 130, 255])) if held > 0 else int(rng.choice([1, 64, 129, 255]))
    churn = int(rng.integers(0, 4))
    hole = int(rng.integers(0, 2)) if held > S else 0
    scale = float(rng.choice([1.0 / np.sqrt(D), 0.05, 0.3]))
    sharp = scale > 0.2          # sharper softmax: outputs of magnitude ~|v| (see the scale 0.7 case above)
    _run_case(A, B, Bc, H, D, T, S, L, held, n_q, n_kc, 20000 + 100 * seed, churn=churn, evict_hole=hole, scale=scale,
              sharp=sharp)


@pytest.mark.parametrize("mode", ["normal", "safe_pass"])
@pytest.mark.parametrize("order", ["rising", "falling", "spike", "steep"])
def test_row_reference_follows_score_jumps_between_tiles(order, mode):
    """Later key tiles score far above (or below) earlier ones.  The fast pass keeps the first tile's maximum as
    the row's reference, which stays exact while exp2 of the difference fits fp32 ("rising", "falling", "spike":
    differences of tens of nats); "steep" rises by hundreds of nats, the row sums overflow and the kernel repeats
    the tile in its safe pass.  In the safe pass a row re-references itself whenever a tile's row sum leaves the
    safe range: several times per row (rising, steep), never after the first tile (falling), once (spike)."""
    from paper_2603_17051_b200 import binding as A
    A.astro_debug_forward_mode(A.FWD_MODE_SAFE_ONLY if mode == "safe_pass" else A.FWD_MODE_NORMAL)
    try:
        _score_jump_case(A, order)
    finally:
        A.astro_debug_forward_mode(A.FWD_MODE_NORMAL)


def _score_jump_case(A, order):
    B, H, D, n_q, n_k = 1, 2, 128, 200, 128 * 6 + 40
    qb = synth.normal_bf16(4101, (B, n_q, H, D)); kb = synth.normal_bf16(4102, (B, n_k, H, D))
    vb = synth.normal_bf16(4103, (B, n_k, H, D)); dob = synth.normal_bf16(4104, (B, n_q, H, D))
    kf = orc.bf16_bits_to_f64(kb)
    tile = np.arange(n_k) // 128
    gain = {"rising": 1.0 + 1.5 * tile, "falling": 10.0 - 1.5 * tile, "spike": np.where(tile == 3, 12.0, 1.0),
            "steep": 1.0 + 12.0 * tile}[order]
    kb = synth.f32_to_bf16_bits((kf * gain[None, :, None, None]).astype(np.float32))   # exact in bf16? re-round
    kf = orc.bf16_bits_to_f64(kb)
    q, k, v, do = (dev_bf16(x) for x in (qb, kb, vb, dob))
    qf, vf, dof = (orc.bf16_bits_to_f64(x) for x in (qb, vb, dob))
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(None, q, k, v, scale)
    A.astro_last_device_status()
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, None, None, kf, vf, scale)
    # near one-hot rows: the output is about one V row, tolerance as in the sharp-softmax case above
    check_fwd(o, lse, o_ref, lse_ref, sharp=True)
    if order != "steep":   # keys 73 times the unit scale are a forward case: bf16 dS then carries ~1.1e-2 into dQ
        g = A.astro_chunk_attn_bwd(None, q, k, v, o, lse, do, scale)
        check_grads(g, orc.chunk_attn_bwd(qf, None, None, kf, vf, dof, scale))


@pytest.mark.parametrize("column", [1, 5, 64 + 2, 64 + 37])
def test_lone_key_far_above_the_first_tile(column):
    """No context; one key of the third tile scores about 100 nats above everything before it, all other keys
    stay near zero.  The key sits on a column whose exponential is taken by the polynomial (column % 16 < 4) or
    by the special-function unit: either way exp2 of the difference to the row's first reference overflows, which
    must be noticed (not wrapped into a small number) and the tile redone with a running reference.  The output
    is then that key's V row and LSE its score."""
    from paper_2603_17051_b200 import binding as A
    B, H, D, n_q, n_k = 1, 2, 128, 140, 128 * 3 + 17
    star = 2 * 128 + column
    rng_q = orc.bf16_bits_to_f64(synth.normal_bf16(4201, (B, n_q, H, D)))
    qb = synth.f32_to_bf16_bits((1.0 + 0.25 * rng_q).astype(np.float32))          # a common direction + noise
    kf = 0.05 * orc.bf16_bits_to_f64(synth.normal_bf16(4202, (B, n_k, H, D)))
    kf[:, star] = 9.0                                                              # score ~ 9 * 128 / sqrt(128) = 102
    kb = synth.f32_to_bf16_bits(kf.astype(np.float32))
    vb = synth.normal_bf16(4203, (B, n_k, H, D)); dob = synth.normal_bf16(4204, (B, n_q, H, D))
    q, k, v, do = (dev_bf16(x) for x in (qb, kb, vb, dob))
    qf, kf, vf, dof = (orc.bf16_bits_to_f64(x) for x in (qb, kb, vb, dob))
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(None, q, k, v, scale)
    A.astro_last_device_status()
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, None, None, kf, vf, scale)
    assert lse_ref.min() > 80.0                                                    # the case is what it claims
    check_fwd(o, lse, o_ref, lse_ref, sharp=True)
    # one-hot rows: dQ and dK vanish (1e-36) and only rounding noise is left of them; dV is the sum of dO at the key
    g = A.astro_chunk_attn_bwd(None, q, k, v, o, lse, do, scale)
    check_grads((None, None, g[2]), orc.chunk_attn_bwd(qf, None, None, kf, vf, dof, scale))


def test_calls_follow_the_callers_stream():
    """Work is enqueued on the stream that is current in torch: results on a side stream match the default one."""
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, T = 2, 2, 128, 40
    cache = A.astro_kvcache_create(B, H, D, T, 1, 3)
    side = torch.cuda.Stream()
    k0, v0 = (dev_bf16(synth.normal_bf16(5100 + i, (B, 3 * T, H, D))) for i in range(2))
    q, kc, vc, do = (dev_bf16(synth.normal_bf16(5110 + i, (B, 150, H, D))) for i in range(4))
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        A.astro_kvcache_append(cache, k0, v0, 3)
        o1, l1 = A.astro_chunk_attn_fwd(cache, q, kc, vc, 0.09)
        g1 = A.astro_chunk_attn_bwd(cache, q, kc, vc, o1, l1, do, 0.09)
    side.synchronize()
    o2, l2 = A.astro_chunk_attn_fwd(cache, q, kc, vc, 0.09)
    g2 = A.astro_chunk_attn_bwd(cache, q, kc, vc, o2, l2, do, 0.09)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    for a, b in zip(g1, g2):
        assert torch.equal(a, b)


def test_many_samples_one_head():
    """Grid dimensions: a batch of 70 samples with a single head, shared and per-sample caches."""
    from paper_2603_17051_b200 import binding as A
    for Bc in (70, 1):
        _run_case(A, B=70, Bc=Bc, H=1, D=64, T=8, S=1, L=2, held=3, n_q=20, n_kc=9, seed=5200 + Bc)


def test_zero_scale_gives_uniform_attention():
    """scale = 0: every key gets the same weight, O is the mean of all values, LSE = ln(number of keys)."""
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, T = 1, 2, 128, 50
    cache = A.astro_kvcache_create(B, H, D, T, 0, 4)
    kx, vx = (dev_bf16(synth.normal_bf16(5300 + i, (B, 4 * T, H, D))) for i in range(2))
    A.astro_kvcache_append(cache, kx, vx, 4)
    q, kc, vc, do = (dev_bf16(synth.normal_bf16(5310 + i, (B, 140, H, D))) for i in range(4))
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, 0.0)
    A.astro_last_device_status()
    mean_v = torch.cat([vx, vc], dim=1).float().mean(dim=1, keepdim=True)
    assert (o.float() - mean_v).abs().max() < 1e-2
    assert (lse - float(np.log(4 * T + 140))).abs().max() < 1e-3
    dq, dk, dv = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, 0.0)
    A.astro_last_device_status()
    assert dq.float().abs().max() == 0 and dk.float().abs().max() == 0          # both carry the factor scale
    expect_dv = do.float().sum(dim=1, keepdim=True) / (4 * T + 140)
    assert (dv.float() - expect_dv).abs().max() < 2e-2


def test_pair_kernel_reports_rows_that_need_the_safe_pass():
    """The CTA-pair kernel keeps one reference per row; a key 100 nats above it overflows exp2 and must be reported."""
    from paper_2603_17051_b200 import binding as A
    B, H, D, n_q, n_k = 1, 1, 128, 130, 128 * 2 + 9
    qb = synth.f32_to_bf16_bits(np.ones((B, n_q, H, D), dtype=np.float32))
    kf = np.zeros((B, n_k, H, D)); kf[:, 128 + 70] = 9.0
    q, k, v = dev_bf16(qb), dev_bf16(synth.f32_to_bf16_bits(kf.astype(np.float32))), dev_bf16(synth.normal_bf16(4303, (B, n_k, H, D)))
    A.astro_debug_pair_flag()
    A.astro_debug_forward_mode(A.FWD_MODE_PAIR)
    try:
        A.astro_chunk_attn_fwd(None, q, k, v, 1.0 / np.sqrt(D))
        A.astro_last_device_status()
        assert A.astro_debug_pair_flag() == 1
        A.astro_chunk_attn_fwd(None, q, k[:, :128].contiguous(), v[:, :128].contiguous(), 1.0 / np.sqrt(D))
        assert A.astro_debug_pair_flag() == 0
    finally:
        A.astro_debug_forward_mode(A.FWD_MODE_NORMAL)


@pytest.mark.parametrize("mode", [0, 2])
def test_group_of_24_candidates_on_one_shared_prefix(mode):
    """Clip-level group-wise sampling at full size: G = 24 candidate chunks (4680 queries each, 12 heads) decode
    against ONE frozen prefix of 18 frames held once (cache_batch = 1); sampled rows of three candidates against
    the oracle, in the normal kernel and in the CTA-pair kernel."""
    from paper_2603_17051_b200 import binding as A
    w = synth.LAYER_FWD
    G, H, D, T, M = 24, w.heads, w.head_dim, w.tokens_per_frame, w.chunk_tokens
    cache, model = _fill(A, 1, H, D, T, w.sink_frames, w.window_frames, w.held_frames, synth.tensor_seed(6, 0), churn=1)
    bits = [synth.normal_bf16(synth.tensor_seed(6, 50 + i), (G, M, H, D)) for i in range(3)]
    q, kc, vc = (dev_bf16(x) for x in bits)
    A.astro_debug_pair_flag()
    A.astro_debug_forward_mode(mode)
    try:
        o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, w.scale)
        A.astro_last_device_status()
        assert A.astro_debug_pair_flag() == 0
    finally:
        A.astro_debug_forward_mode(0)
    mk, mv = model.export()
    rows = _sample_rows(M, 24, np.random.default_rng(6))
    for (b, h) in ((0, 0), (11, 5), (23, 11)):
        sl = lambda x: orc.bf16_bits_to_f64(x[b:b + 1, :, h:h + 1, :])
        kx, vx = orc.bf16_bits_to_f64(mk[:, :, h:h + 1, :]), orc.bf16_bits_to_f64(mv[:, :, h:h + 1, :])
        o_ref, lse_ref = orc.chunk_attn_fwd(sl(bits[0])[:, rows], kx, vx, sl(bits[1]), sl(bits[2]), w.scale)
        check_fwd(o[b:b + 1, rows, h:h + 1], lse[b:b + 1, h:h + 1][:, :, rows], o_ref, lse_ref, tag="b%d h%d" % (b, h))


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("n_k", [100, 200, 3 * 128, 5 * 128 + 9])
def test_more_work_units_than_sms_with_few_key_tiles(n_k, D):
    """240 (query tile, head, sample) units of 1, 2, 3 or 6 key tiles each: every CTA walks over two of them, so
    the S look-ahead, the K/V rings and the two Q buffers all cross unit boundaries, with units shorter than the
    look-ahead itself; the last query tile is ragged.  At head_dim 64 only half of the epilogue warps stage Q."""
    from paper_2603_17051_b200 import binding as A
    B, H, n_q = 3, 20, 3 * 128 + 16
    qb = synth.normal_bf16(5101, (B, n_q, H, D)); kb = synth.normal_bf16(5102, (B, n_k, H, D))
    vb = synth.normal_bf16(5103, (B, n_k, H, D))
    q, k, v = (dev_bf16(x) for x in (qb, kb, vb))
    qf, kf, vf = (orc.bf16_bits_to_f64(x) for x in (qb, kb, vb))
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(None, q, k, v, scale)
    A.astro_last_device_status()
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, None, None, kf, vf, scale)
    check_fwd(o, lse, o_ref, lse_ref)


def test_some_units_of_a_cta_need_the_safe_pass():
    """444 units of three key tiles; in heads 1 and 4 the keys of the later tiles are scaled up so far that the rows'
    sums overflow against their first-tile reference.  Only the units of those heads are redone by the safe pass;
    they sit between units of other heads in the walk of one CTA."""
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, n_q, n_k = 2, 6, 128, 37 * 128 - 50, 3 * 128
    qb = synth.normal_bf16(5201, (B, n_q, H, D)); kb = synth.normal_bf16(5202, (B, n_k, H, D))
    vb = synth.normal_bf16(5203, (B, n_k, H, D))
    kf = orc.bf16_bits_to_f64(kb)
    gain = 1.0 + 30.0 * (np.arange(n_k) // 128)
    for h in (1, 4):
        kf[:, :, h] *= gain[None, :, None]
    kb = synth.f32_to_bf16_bits(kf.astype(np.float32))
    q, k, v = (dev_bf16(x) for x in (qb, kb, vb))
    qf, kf, vf = (orc.bf16_bits_to_f64(x) for x in (qb, kb, vb))
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(None, q, k, v, scale)
    A.astro_last_device_status()
    rows = np.concatenate([np.arange(0, n_q, 97), np.arange(n_q - 40, n_q)])   # sampled rows and the ragged tile
    o_ref, lse_ref = orc.chunk_attn_fwd(qf[:, rows], None, None, kf, vf, scale)
    pick = torch.from_numpy(rows).to(o.device)
    check_fwd(o[:, pick], lse[:, :, pick], o_ref, lse_ref, sharp=True)
