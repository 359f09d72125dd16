"""GPU parity of the fused NFT policy loss + selective KL + gradient against the fp64 oracle."""
import numpy as np
import pytest

from helpers import dev_bf16, f64, rel_l2
from oracle import nft_loss as nft
from oracle.rolling_attn import bf16_bits_to_f64
from paper_2603_17051_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,E,beta,with_ref", [(3, 8, 1.0, True), (2, 1000, 0.1, True), (5, 4096 * 3 + 8, 1.0, False),
                                               (24, 3 * 16 * 60 * 104, 1.0, True)])
def test_nft_loss_parity(B, E, beta, with_ref):
    import torch
    from paper_2603_17051_b200 import binding as A
    bits = [synth.normal_bf16(synth.tensor_seed(6, 10 * B + i), (B, E)) for i in range(4)]
    vt, vo, vr, tg = (dev_bf16(x) for x in bits)
    f = [bf16_bits_to_f64(x) for x in bits]
    rng = np.random.default_rng(B)
    r = rng.uniform(0, 1, B).astype(np.float32); wp = rng.uniform(0.1, 1, B).astype(np.float32) / E
    wk = (rng.integers(0, 2, B) * 1e-4 / max(E, 1)).astype(np.float32)
    tr, twp, twk = (torch.from_numpy(x).cuda() for x in (r, wp, wk))
    policy, kl, g = A.astro_nft_loss(vt, vo, vr if with_ref else None, tg, tr, beta, w_policy=twp,
                                     w_kl=twk if with_ref else None)
    p_ref, k_ref = nft.nft_loss(f[0], f[1], f[2], f[3], r.astype(np.float64), beta)
    g_ref = nft.nft_loss_grad(f[0], f[1], f[2], f[3], r.astype(np.float64), beta, wp.astype(np.float64),
                              wk.astype(np.float64) if with_ref else np.zeros(B))
    # fp32 sums of up to 3e5 positive terms: relative 1e-4; gradient rounded to bf16: relative L2 1e-2
    assert np.allclose(f64(policy), p_ref, rtol=1e-4)
    if with_ref:
        assert np.allclose(f64(kl), k_ref, rtol=1e-4)
    else:
        assert kl is None
    assert rel_l2(f64(g), g_ref) <= 1e-2
    # loss only (no gradient buffer) gives the same losses
    p2, _, g2 = A.astro_nft_loss(vt, vo, vr if with_ref else None, tg, tr, beta, grad=False)
    assert g2 is None and np.allclose(f64(p2), p_ref, rtol=1e-4)


def test_nft_loss_argument_checks():
    import torch
    from paper_2603_17051_b200 import binding as A
    x = torch.zeros((2, 12), dtype=torch.bfloat16, device="cuda")      # 12 is not a multiple of 8
    r = torch.zeros(2, dtype=torch.float32, device="cuda")
    with pytest.raises(A.AstroError) as e:
        A.astro_nft_loss(x, x, x, x, r, 1.0)
    assert e.value.status == 2
