"""GPU parity of the ring cache (append / evict / export) against the oracle's deque model: bit-exact."""
import numpy as np
import pytest

from helpers import dev_bf16, host_bits
from oracle import rolling_attn as orc
from paper_2603_17051_b200 import synth

pytestmark = pytest.mark.gpu


def _both_export_equal(A, cache, model):
    ke, ve = A.astro_kvcache_export(cache)
    mk, mv = model.export()
    if mk is None:
        assert ke.shape[1] == 0
        return
    assert np.array_equal(host_bits(ke), mk)
    assert np.array_equal(host_bits(ve), mv)


@pytest.mark.parametrize("Bc,H,D,T,S,L", [(1, 2, 64, 16, 0, 6), (2, 3, 128, 20, 3, 5), (1, 1, 64, 7, 1, 1)])
def test_random_append_evict_sequences_are_bit_exact(Bc, H, D, T, S, L):
    from paper_2603_17051_b200 import binding as A
    rng = np.random.default_rng(1234 + S + L)
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L)
    model = orc.RollingKVCache(S, L)
    seed = 5000
    for step in range(60):
        sink, win, seen = A.astro_kvcache_query(cache)
        assert (sink, win, seen) == (len(model.sink_k), len(model.win_k), model.frames_seen)
        assert sink + win <= S + L
        room = S + L - sink - win
        if rng.random() < 0.4 and win > 0:
            n = int(rng.integers(1, win + 1))
            A.astro_kvcache_evict(cache, n); model.evict(n)
        elif room > 0:
            f = int(rng.integers(1, room + 1))
            kb = synth.normal_bf16(seed, (Bc, f * T, H, D)); vb = synth.normal_bf16(seed + 1, (Bc, f * T, H, D))
            seed += 2
            A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), f); model.append(kb, vb, T)
        else:
            with pytest.raises(A.AstroError) as e:
                A.astro_kvcache_append(cache, dev_bf16(np.zeros((Bc, T, H, D), np.uint16)),
                                       dev_bf16(np.zeros((Bc, T, H, D), np.uint16)), 1)
            assert e.value.status == 4
            A.astro_kvcache_evict(cache, 1); model.evict(1)
        _both_export_equal(A, cache, model)
    with pytest.raises(A.AstroError) as e:
        A.astro_kvcache_evict(cache, L + 1)
    assert e.value.status == 5
    A.astro_kvcache_reset(cache); model.reset()
    assert A.astro_kvcache_query(cache) == (0, 0, 0)


def test_sink_frames_survive_eighty_chunks_and_memory_is_constant():
    """Structural statements of the rolling cache: sink kept for good, window = most recent frames,
    resident storage independent of the video length."""
    from paper_2603_17051_b200 import binding as A
    Bc, H, D, T, S, L, c = 1, 2, 64, 16, 3, 12, 3
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L)
    ptrs = (cache.k_storage.data_ptr(), cache.v_storage.data_ptr(), cache.k_storage.numel())
    model = orc.RollingKVCache(S, L)
    first_sink = None
    for n in range(80):
        over = model.held() - (S + L - c)
        if over > 0:
            A.astro_kvcache_evict(cache, over); model.evict(over)
        kb = synth.normal_bf16(7000 + 2 * n, (Bc, c * T, H, D)); vb = synth.normal_bf16(7001 + 2 * n, (Bc, c * T, H, D))
        A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), c); model.append(kb, vb, T)
        if first_sink is None:
            first_sink = kb[:, :S * T].copy()
        sink, win, seen = A.astro_kvcache_query(cache)
        assert sink + win <= S + L and seen == (n + 1) * c
    ke, ve = A.astro_kvcache_export(cache)
    assert np.array_equal(host_bits(ke)[:, :S * T], first_sink)
    _both_export_equal(A, cache, model)
    assert ptrs == (cache.k_storage.data_ptr(), cache.v_storage.data_ptr(), cache.k_storage.numel())


def test_append_in_pieces_larger_than_one_launch():
    from paper_2603_17051_b200 import binding as A
    Bc, H, D, T, S, L = 2, 1, 64, 3, 2, 40
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L)
    model = orc.RollingKVCache(S, L)
    kb = synth.normal_bf16(8000, (Bc, 42 * T, H, D)); vb = synth.normal_bf16(8001, (Bc, 42 * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), 42); model.append(kb, vb, T)
    _both_export_equal(A, cache, model)


def test_saved_storage_and_state_resume_on_a_new_handle():
    """Checkpoint/resume: clone the storage bytes, carry the state record over, continue streaming."""
    from paper_2603_17051_b200 import binding as A
    Bc, H, D, T, S, L = 2, 2, 64, 9, 2, 5
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L)
    model = orc.RollingKVCache(S, L)
    seed = 9100
    for n in range(9):                                       # fill, then churn so the ring head is mid-way
        if model.held() == S + L:
            A.astro_kvcache_evict(cache, 2); model.evict(2)
        kb = synth.normal_bf16(seed, (Bc, T, H, D)); vb = synth.normal_bf16(seed + 1, (Bc, T, H, D)); seed += 2
        A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), 1); model.append(kb, vb, T)
    state = A.astro_kvcache_get_state(cache)
    resumed = A.astro_kvcache_create(Bc, H, D, T, S, L, k_storage=cache.k_storage.clone(),
                                     v_storage=cache.v_storage.clone())
    A.astro_kvcache_set_state(resumed, state)
    _both_export_equal(A, resumed, model)
    A.astro_kvcache_evict(resumed, 1); model.evict(1)
    kb = synth.normal_bf16(seed, (Bc, T, H, D)); vb = synth.normal_bf16(seed + 1, (Bc, T, H, D))
    A.astro_kvcache_append(resumed, dev_bf16(kb), dev_bf16(vb), 1); model.append(kb, vb, T)
    _both_export_equal(A, resumed, model)
    assert A.astro_kvcache_query(resumed)[2] == model.frames_seen


def test_cache_storage_canaries_are_untouched():
    """Appends at every ring position write inside the bound storage only (padding on both sides stays intact)."""
    import torch
    from paper_2603_17051_b200 import binding as A
    Bc, H, D, T, S, L = 2, 3, 128, 11, 2, 3
    nbytes = A.astro_kvcache_storage_bytes(Bc, H, D, T, S, L)
    pad = 4096
    bufs = [torch.full((nbytes + 2 * pad,), 0x5A, dtype=torch.uint8, device="cuda") for _ in range(2)]
    cache = A.astro_kvcache_create(Bc, H, D, T, S, L, k_storage=bufs[0][pad:pad + nbytes],
                                   v_storage=bufs[1][pad:pad + nbytes])
    model = orc.RollingKVCache(S, L)
    for n in range(12):
        if model.held() == S + L:
            A.astro_kvcache_evict(cache, 1); model.evict(1)
        kb = synth.normal_bf16(9300 + 2 * n, (Bc, T, H, D)); vb = synth.normal_bf16(9301 + 2 * n, (Bc, T, H, D))
        A.astro_kvcache_append(cache, dev_bf16(kb), dev_bf16(vb), 1); model.append(kb, vb, T)
    _both_export_equal(A, cache, model)
    for b in bufs:
        assert (b[:pad] == 0x5A).all() and (b[-pad:] == 0x5A).all()
