"""CPU oracle for the forward-process policy loss with selective KL.  TEST INFRASTRUCTURE ONLY.

fp64 numpy restatement of Eq. 1 (implicit positive / negative velocities), Eq. 2 (policy loss) and the
selective KL term of Sec. 3.4 / Algorithm 2, per sample, plus the gradient with respect to the current
policy's velocity.  Shares nothing with the CUDA path.

Conventions (the paper leaves the reduction open): ||.||^2 is the plain sum of squares over a sample's
elements; per-sample values are returned and the caller combines them (mean over the batch, mask and
lambda_KL / |M| for the KL term).  The gradient is that of sum_i (w_policy_i * policy_i + w_kl_i * kl_i).

Pins (tests/test_oracle_pins_nft.py): beta = 0 and v_theta = v_old collapse both branches onto v_old;
scalar closed form; the symmetry (r, beta) -> (1 - r, -beta); finite differences of the gradient;
the KL term against numpy's own norm.
"""
from __future__ import annotations

import numpy as np


def nft_loss(v_theta, v_old, v_ref, v_target, r_tilde, beta: float):
    """Per-sample policy loss (Eq. 2) and squared distance to the reference policy.

    v_* and v_target: [B, E]; r_tilde: [B] in [0, 1].  Returns (policy[B], kl[B])."""
    v_theta = np.asarray(v_theta, np.float64); v_old = np.asarray(v_old, np.float64)
    v_ref = np.asarray(v_ref, np.float64); v_target = np.asarray(v_target, np.float64)
    r = np.asarray(r_tilde, np.float64)
    v_pos = (1.0 - beta) * v_old + beta * v_theta            # Eq. 1
    v_neg = (1.0 + beta) * v_old - beta * v_theta
    policy = r * ((v_pos - v_target) ** 2).sum(axis=1) + (1.0 - r) * ((v_neg - v_target) ** 2).sum(axis=1)  # Eq. 2
    kl = ((v_theta - v_ref) ** 2).sum(axis=1)
    return policy, kl


def nft_loss_grad(v_theta, v_old, v_ref, v_target, r_tilde, beta: float, w_policy, w_kl):
    """d/d v_theta of sum_i (w_policy_i * policy_i + w_kl_i * kl_i), shape [B, E]."""
    v_theta = np.asarray(v_theta, np.float64); v_old = np.asarray(v_old, np.float64)
    v_ref = np.asarray(v_ref, np.float64); v_target = np.asarray(v_target, np.float64)
    r = np.asarray(r_tilde, np.float64)[:, None]
    wp = np.asarray(w_policy, np.float64)[:, None]; wk = np.asarray(w_kl, np.float64)[:, None]
    v_pos = (1.0 - beta) * v_old + beta * v_theta
    v_neg = (1.0 + beta) * v_old - beta * v_theta
    g_policy = 2.0 * beta * (r * (v_pos - v_target) - (1.0 - r) * (v_neg - v_target))
    g_kl = 2.0 * (v_theta - v_ref)
    return wp * g_policy + wk * g_kl
