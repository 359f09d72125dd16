"""Backward without caller scratch (astro_chunk_attn_bwd_static), for callers that cannot allocate device
memory: a loop whose allocator is frozen after warm-up, code running inside another framework's pool.

Collected last on purpose, so that a run stopping at the first failure has already run everything else.
The entry point is called through the C ABI twice in a row (the shared device array keeps the first call's
contents, the second call must not care) and compared with astro_chunk_attn_bwd on the same inputs and with the
fp64 oracle."""
import numpy as np
import pytest

from helpers import GRAD_REL_L2, check_grads, dev_bf16, f64, rel_l2
from oracle import rolling_attn as orc
from paper_2603_17051_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_scratch_backward_matches_workspace_backward_twice():
    import torch
    from paper_2603_17051_b200 import binding as A
    H, D, T, S, L, held = 3, 128, 40, 1, 5, 5
    cache = A.astro_kvcache_create(1, H, D, T, S, L)
    kxb, vxb = synth.normal_bf16(9001, (1, held * T, H, D)), synth.normal_bf16(9002, (1, held * T, H, D))
    A.astro_kvcache_append(cache, dev_bf16(kxb), dev_bf16(vxb), held)
    kx, vx = orc.bf16_bits_to_f64(kxb), orc.bf16_bits_to_f64(vxb)
    for call, (B, n_q, n_kc) in enumerate(((2, 300, 300), (1, 170, 90))):   # second call: smaller problem
        qb, dob = (synth.normal_bf16(9010 + 10 * call + i, (B, n_q, H, D)) for i in range(2))
        kcb, vcb = (synth.normal_bf16(9015 + 10 * call + i, (B, n_kc, H, D)) for i in range(2))
        q, do, kc, vc = (dev_bf16(x) for x in (qb, dob, kcb, vcb))
        o, lse = A.astro_chunk_attn_fwd(cache, q, kc, vc, 0.09)
        ref = A.astro_chunk_attn_bwd(cache, q, kc, vc, o, lse, do, 0.09)
        dq, dk, dv = torch.zeros_like(q), torch.zeros_like(kc), torch.zeros_like(vc)
        A.astro_chunk_attn_bwd_static(cache, q, kc, vc, o, lse, do, 0.09, dq, dk, dv)
        A.astro_last_device_status()
        for got, want, name in zip((dq, dk, dv), ref, ("dQ", "dK", "dV")):
            e = rel_l2(f64(got), f64(want))
            assert e <= GRAD_REL_L2, "call %d %s rel-L2 %.3e" % (call, name, e)
        qf, dof, kf, vf = (orc.bf16_bits_to_f64(x) for x in (qb, dob, kcb, vcb))
        check_grads((dq, dk, dv), orc.chunk_attn_bwd(qf, kx, vx, kf, vf, dof, 0.09), tag="call %d vs oracle" % call)


def test_static_scratch_backward_rejects_sizes_beyond_its_array():
    import torch
    from paper_2603_17051_b200 import binding as A
    B, H, D = 1, 2, 64
    n_q = A.BWD_STATIC_MAX_ROWS // (B * H) + 1
    q = torch.zeros((B, n_q, H, D), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((B, 8, H, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((B, H, n_q), dtype=torch.float32, device="cuda")
    with pytest.raises(A.AstroError) as e:
        A.astro_chunk_attn_bwd_static(None, q, kc, kc, q, lse, q, 0.1, torch.empty_like(q), torch.empty_like(kc),
                                      torch.empty_like(kc))
    assert e.value.status == 4
