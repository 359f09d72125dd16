"""GPU parity of the backward's three stage calls (delta, dQ, dK/dV) taken one by one through the C ABI, each against
the oracle -- these are the entry points the benchmark times -- and of the window-variant shapes of Tab. S1."""
import numpy as np
import pytest

from helpers import GRAD_REL_L2, check_fwd, check_grads, dev_bf16, f64, host_bits, rel_l2
from oracle import rolling_attn as orc
from paper_2603_17051_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(seed, B, n_q, n_kc, H, D):
    bits = [synth.normal_bf16(seed + i, shp) for i, shp in
            enumerate(((B, n_q, H, D), (B, n_kc, H, D), (B, n_kc, H, D), (B, n_q, H, D)))]
    return bits, [dev_bf16(x) for x in bits], [orc.bf16_bits_to_f64(x) for x in bits]


@pytest.mark.parametrize("D,Bc", [(128, 2), (64, 1)])
def test_backward_stages_one_by_one_against_the_oracle(D, Bc):
    """delta from the ORACLE's O and dO must match oracle.bwd_delta; dQ and dK/dV are then computed from the
    oracle's own LSE and delta (uploaded as fp32), so each stage is checked on inputs no other GPU stage produced."""
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, T, S, L, held, n_q, n_kc = 2, 3, 50, 1, 6, 6, 300, 170
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L)
    model = orc.RollingKVCache(S, L)
    kb = synth.normal_bf16(8101, (Bc, held * T, H, D)); vb = synth.normal_bf16(8102, (Bc, held * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), held); model.append(kb, vb, T)
    A.astro_kvcache_evict(cache, 2); model.evict(2)                       # a hole: two cache ranges
    bits, (q, kc, vc, do), (qf, kf, vf, dof) = _inputs(8110, B, n_q, n_kc, H, D)
    mk, mv = model.export()
    kx, vx = orc.bf16_bits_to_f64(mk), orc.bf16_bits_to_f64(mv)
    scale = 1.0 / np.sqrt(D)
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, kx, vx, kf, vf, scale)
    dq_ref, dk_ref, dv_ref = orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, scale)
    # stage 1: delta = rowsum(dO * O) on the bf16-rounded oracle output
    o_bits = synth.f32_to_bf16_bits(o_ref.astype(np.float32))
    delta = A.astro_chunk_attn_bwd_delta(dev_bf16(o_bits), do)
    delta_ref = orc.bwd_delta(orc.bf16_bits_to_f64(o_bits), dof)          # [B, H, n_q]
    assert np.abs(f64(delta) - delta_ref).max() <= 1e-4 * max(1.0, np.abs(delta_ref).max())
    # stages 2 and 3 from the oracle's statistics
    lse_d = torch.from_numpy(np.ascontiguousarray(lse_ref, dtype=np.float32)).cuda()
    delta_d = torch.from_numpy(np.ascontiguousarray(orc.bwd_delta(o_ref, dof), dtype=np.float32)).cuda()
    dq = A.astro_chunk_attn_bwd_dq(cache, q, kc, vc, lse_d, delta_d, do, scale)
    dk, dv = A.astro_chunk_attn_bwd_dkv(q, kc, vc, lse_d, delta_d, do, scale)
    A.astro_last_device_status()
    check_grads((dq, dk, dv), (dq_ref, dk_ref, dv_ref))


def test_dq_stage_without_chunk_keys_and_dkv_stage_without_cache():
    """dQ over cached keys only (n_kc = 0), and dK/dV with no cache involved at all."""
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D, T, n_q, n_kc = 1, 2, 128, 64, 200, 140
    cache = A.astro_kvcache_create(1, H, D, T, 0, 4)
    model = orc.RollingKVCache(0, 4)
    kb = synth.normal_bf16(8201, (1, 3 * T, H, D)); vb = synth.normal_bf16(8202, (1, 3 * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), 3); model.append(kb, vb, T)
    bits, (q, kc, vc, do), (qf, kf, vf, dof) = _inputs(8210, B, n_q, n_kc, H, D)
    kx, vx = (orc.bf16_bits_to_f64(x) for x in model.export())
    empty = np.zeros((B, 0, H, D))
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, kx, vx, empty, empty, 0.1)
    dq_ref, _, _ = orc.chunk_attn_bwd(qf, kx, vx, empty, empty, dof, 0.1)
    dev32 = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    dq = A.astro_chunk_attn_bwd_dq(cache, q, None, None, dev32(lse_ref), dev32(orc.bwd_delta(o_ref, dof)), do, 0.1)
    A.astro_last_device_status()
    check_grads((dq, None, None), (dq_ref, None, None))
    o_ref, lse_ref = orc.chunk_attn_fwd(qf, None, None, kf, vf, 0.1)
    _, dk_ref, dv_ref = orc.chunk_attn_bwd(qf, None, None, kf, vf, dof, 0.1)
    dk, dv = A.astro_chunk_attn_bwd_dkv(q, kc, vc, dev32(lse_ref), dev32(orc.bwd_delta(o_ref, dof)), do, 0.1)
    A.astro_last_device_status()
    check_grads((None, dk, dv), (None, dk_ref, dv_ref))


def _sample_rows(n_q, n_rand, rng):
    tail = np.arange((n_q // 128) * 128, n_q)
    return np.unique(np.concatenate([rng.choice(n_q, n_rand, replace=False), tail, [0, 127, 128]]))


@pytest.mark.parametrize("total_frames", [21, 15])
def test_per_frame_chunk_against_the_window_presets(total_frames):
    """Tab. S1 presets with per-frame chunks: one frame of 1560 queries (12 full query tiles and a ragged one of 24
    rows) attends to 20 or 14 held frames (3 sink + window) plus itself, 12 heads, batch 2; sampled rows and the
    whole ragged tile against the oracle."""
    from paper_2603_17051_b200 import binding as A
    B, H, D, T, S = 2, 12, 128, 1560, 3
    held = total_frames - 1
    cache = A.astro_kvcache_create(B, H, D, T, S, total_frames - S)
    model = orc.RollingKVCache(S, total_frames - S)
    kb = synth.normal_bf16(synth.tensor_seed(7, total_frames), (B, held * T, H, D))
    vb = synth.normal_bf16(synth.tensor_seed(7, total_frames + 100), (B, held * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), held); model.append(kb, vb, T)
    bits = [synth.normal_bf16(synth.tensor_seed(7, 200 + total_frames + i), (B, T, H, D)) for i in range(3)]
    q, kc, vc = (dev_bf16(x) for x in bits)
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, scale)
    A.astro_last_device_status()
    mk, mv = model.export()
    rows = _sample_rows(T, 40, np.random.default_rng(total_frames))
    for (b, h) in ((0, 2), (1, 9)):
        sl = lambda x: orc.bf16_bits_to_f64(x[b:b + 1, :, h:h + 1, :])
        o_ref, lse_ref = orc.chunk_attn_fwd(sl(bits[0])[:, rows], sl(mk), sl(mv), sl(bits[1]), sl(bits[2]), scale)
        check_fwd(o[b:b + 1, rows, h:h + 1], lse[b:b + 1, h:h + 1][:, :, rows], o_ref, lse_ref, tag="b%d h%d" % (b, h))
    # the frame joins the cache; the oldest window frame leaves first (capacity counts the chunk)
    A.astro_kvcache_evict(cache, 1); model.evict(1)
    A.astro_kvcache_append(cache, kc, vc, 1); model.append(bits[1], bits[2], T)
    ke, ve = A.astro_kvcache_export(cache)
    mk, mv = model.export()
    assert np.array_equal(host_bits(ke), mk) and np.array_equal(host_bits(ve), mv)


def test_prompt_switch_rebuilds_the_cache():
    """Multi-prompt generation (Tab. 3): when the prompt changes the text-conditioned cache is rebuilt -- reset, the
    first S frames appended afterwards become the new sink, the window refills -- while the storage and the handle
    stay.  Cache contents bit-exact before and after the switch; attention after it sees only the new frames."""
    from paper_2603_17051_b200 import binding as A
    B, H, D, T, S, L, c = 2, 3, 128, 96, 2, 5, 2
    cache = A.astro_kvcache_create(B, H, D, T, S, L)
    model = orc.RollingKVCache(S, L)
    seed = 8400
    def stream(n_chunks):
        nonlocal seed
        for _ in range(n_chunks):
            over = model.held() - (S + L - c)
            if over > 0:
                A.astro_kvcache_evict(cache, over); model.evict(over)
            kb = synth.normal_bf16(seed, (B, c * T, H, D)); vb = synth.normal_bf16(seed + 1, (B, c * T, H, D))
            seed += 2
            A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), c); model.append(kb, vb, T)
    stream(5)                                             # first prompt: ring wrapped, head in the middle
    assert A.astro_kvcache_query(cache) == (2, 5, 10)
    A.astro_kvcache_reset(cache); model.reset()            # prompt switch
    assert A.astro_kvcache_query(cache) == (0, 0, 0)
    stream(2)                                             # re-seed: S sink frames + 2 window frames of the new prompt
    ke, ve = A.astro_kvcache_export(cache)
    mk, mv = model.export()
    assert np.array_equal(host_bits(ke), mk) and np.array_equal(host_bits(ve), mv)
    assert A.astro_kvcache_query(cache) == (2, 2, 4)
    bits, (q, kc, vc, do), (qf, kf, vf, dof) = _inputs(8450, B, c * T, c * T, H, D)
    scale = 1.0 / np.sqrt(D)
    o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, scale)
    g = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, scale)
    A.astro_last_device_status()
    kx, vx = orc.bf16_bits_to_f64(mk), orc.bf16_bits_to_f64(mv)
    check_fwd(o, lse, *orc.chunk_attn_fwd(qf, kx, vx, kf, vf, scale))
    check_grads(g, orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, scale))
    stream(4)                                             # and the new prompt keeps streaming: sink kept, window slides
    ke, ve = A.astro_kvcache_export(cache)
    mk, mv = model.export()
    assert np.array_equal(host_bits(ke), mk) and np.array_equal(host_bits(ve), mv)
