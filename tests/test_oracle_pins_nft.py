"""Pins for the NFT-loss oracle: closed forms, symmetries and finite differences."""
import numpy as np

from oracle import nft_loss as nft


def rnd(seed, shape):
    return np.random.default_rng(seed).standard_normal(shape)


def test_scalar_closed_form():
    # one sample, one element: v_theta=2, v_old=1, target=0.5, beta=0.5, r=0.25
    # v+ = 0.5*1 + 0.5*2 = 1.5 ; v- = 1.5*1 - 0.5*2 = 0.5 ; loss = 0.25*(1.0)^2 + 0.75*0^2 = 0.25
    p, k = nft.nft_loss([[2.0]], [[1.0]], [[-1.0]], [[0.5]], [0.25], 0.5)
    assert p[0] == 0.25 and k[0] == 9.0
    g = nft.nft_loss_grad([[2.0]], [[1.0]], [[-1.0]], [[0.5]], [0.25], 0.5, [1.0], [0.0])
    assert g[0, 0] == 2 * 0.5 * (0.25 * 1.0 - 0.75 * 0.0)
    # beta = 1 (the paper's default): v+ = v_theta, v- = 2 v_old - v_theta
    p, _ = nft.nft_loss([[2.0]], [[1.0]], [[0.0]], [[0.5]], [1.0], 1.0)
    assert p[0] == (2.0 - 0.5) ** 2
    p, _ = nft.nft_loss([[2.0]], [[1.0]], [[0.0]], [[0.5]], [0.0], 1.0)
    assert p[0] == (0.0 - 0.5) ** 2


def test_collapses_to_old_policy():
    B, E = 3, 40
    vt, vo, vr, tg = rnd(1, (B, E)), rnd(2, (B, E)), rnd(3, (B, E)), rnd(4, (B, E))
    r = np.array([0.1, 0.5, 0.9])
    base = ((vo - tg) ** 2).sum(1)
    p0, _ = nft.nft_loss(vt, vo, vr, tg, r, 0.0)                 # beta = 0: both branches are v_old
    assert np.allclose(p0, base, atol=1e-12)
    assert np.abs(nft.nft_loss_grad(vt, vo, vr, tg, r, 0.0, np.ones(B), np.zeros(B))).max() == 0.0
    p1, _ = nft.nft_loss(vo, vo, vr, tg, r, 0.7)                 # v_theta = v_old: same, whatever r is
    assert np.allclose(p1, base, atol=1e-12)


def test_symmetry_between_positive_and_negative_branch():
    B, E = 2, 30
    vt, vo, vr, tg = rnd(5, (B, E)), rnd(6, (B, E)), rnd(7, (B, E)), rnd(8, (B, E))
    r = np.array([0.2, 0.8])
    a, _ = nft.nft_loss(vt, vo, vr, tg, r, 0.6)
    b, _ = nft.nft_loss(vt, vo, vr, tg, 1.0 - r, -0.6)           # swapping the branches swaps their weights
    assert np.allclose(a, b, atol=1e-12)


def test_kl_term_is_squared_distance_and_independent_of_the_rest():
    B, E = 2, 25
    vt, vo, vr, tg = rnd(9, (B, E)), rnd(10, (B, E)), rnd(11, (B, E)), rnd(12, (B, E))
    _, k = nft.nft_loss(vt, vo, vr, tg, [0.3, 0.4], 1.0)
    assert np.allclose(k, np.linalg.norm(vt - vr, axis=1) ** 2, atol=1e-12)
    _, k2 = nft.nft_loss(vt, vo * 3, vr, tg + 1, [0.9, 0.0], 0.1)
    assert np.array_equal(k, k2)


def test_gradient_matches_central_finite_differences():
    B, E = 2, 6
    vt, vo, vr, tg = rnd(13, (B, E)), rnd(14, (B, E)), rnd(15, (B, E)), rnd(16, (B, E))
    r, wp, wk, beta = np.array([0.3, 0.85]), np.array([0.5, 2.0]), np.array([0.0, 0.25]), 0.8
    g = nft.nft_loss_grad(vt, vo, vr, tg, r, beta, wp, wk)

    def total(x):
        p, k = nft.nft_loss(x, vo, vr, tg, r, beta)
        return float((wp * p + wk * k).sum())
    h = 1e-6
    for i in range(B):
        for e in range(E):
            x = vt.copy(); x[i, e] += h; lp = total(x)
            x[i, e] -= 2 * h; lm = total(x)
            assert abs((lp - lm) / (2 * h) - g[i, e]) < 1e-6
