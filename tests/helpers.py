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


def check_fwd(o, lse, o_ref, lse_ref, tag=""):
    d = np.abs(f64(o) - o_ref)
    assert d.max() <= O_MAX_ABS, "%s O max-abs %.3e" % (tag, d.max())
    assert d.mean() <= O_MEAN_ABS, "%s O mean-abs %.3e" % (tag, d.mean())
    dl = np.abs(f64(lse) - lse_ref)
    assert dl.max() <= LSE_ABS, "%s LSE abs %.3e" % (tag, dl.max())


def check_grads(got, ref, tag=""):
    for g, r, name in zip(got, ref, ("dQ", "dK", "dV")):
        if g is None:
            continue
        e = rel_l2(f64(g), r)
        assert e <= GRAD_REL_L2, "%s %s rel-L2 %.3e" % (tag, name, e)
