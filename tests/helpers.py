"""Shared helpers of the GPU parity tests: host<->device marshalling and oracle-side views."""
import numpy as np


def dev_bf16(bits, device="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def host_bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f64(t):
    return t.double().cpu().numpy()


def rel_l2(got, ref):
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


# Tolerances of the parity bar: O max-abs 1e-2 and mean-abs 1e-3; LSE abs 1e-3; gradients relative L2 1e-2.
O_MAX_ABS, O_MEAN_ABS, LSE_ABS, GRAD_REL_L2 = 1e-2, 1e-3, 1e-3, 1e-2


def bf16_ulp(x):
    """Spacing of bf16 numbers (8 significant bits) at the magnitude of x; 0 where x is 0."""
    a = np.abs(np.asarray(x, dtype=np.float64))
    out = np.zeros_like(a)
    nz = a > 0
    out[nz] = np.exp2(np.floor(np.log2(a[nz])) - 7)
    return out


def check_fwd(o, lse, o_ref, lse_ref, tag="", sharp=False):
    """O within max-abs 1e-2 and mean-abs 1e-3, LSE within 1e-3.  With `sharp` (near one-hot softmax rows, where
    the output is about one V row of magnitude up to ~4.5) every element is still held to 1e-2 plus the rounding
    that no bf16 output can avoid: half a bf16 ulp of its own reference value (a quarter ulp in the mean)."""
    d = np.abs(f64(o) - o_ref)
    if sharp:
        ulp = bf16_ulp(o_ref)
        excess = d - (O_MAX_ABS + 0.5 * ulp)
        assert excess.max() <= 0, "%s O error exceeds 1e-2 + half a bf16 ulp by %.3e" % (tag, excess.max())
        bound = O_MEAN_ABS + 0.25 * ulp.mean()
        assert d.mean() <= bound, "%s O mean-abs %.3e > %.3e" % (tag, d.mean(), bound)
    else:
        assert d.max() <= O_MAX_ABS, "%s O max-abs %.3e" % (tag, d.max())
        assert d.mean() <= O_MEAN_ABS, "%s O mean-abs %.3e" % (tag, d.mean())
    dl = np.abs(f64(lse) - lse_ref)
    assert dl.max() <= LSE_ABS, "%s LSE abs %.3e" % (tag, dl.max())


def check_grads(got, ref, tag=""):
    for g, r, name in zip(got, ref, ("dQ", "dK", "dV")):
        if g is None:
            continue
        # relative L2 with an absolute floor of 1e-6 per element, for gradients that are exactly zero
        # mathematically (a single key: softmax is constant, dQ = dK = 0) where fp32 rounding noise remains
        err = float(np.linalg.norm(f64(g) - r))
        bound = GRAD_REL_L2 * float(np.linalg.norm(r)) + 1e-6 * np.sqrt(r.size)
        assert err <= bound, "%s %s rel-L2 %.3e (err %.3e, bound %.3e)" % (tag, name, rel_l2(f64(g), r), err, bound)
