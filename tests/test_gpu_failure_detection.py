"""Failure detection without a GPU fault: a device-side wait that runs out is reported through the status
word, the kernel ends normally and the context stays usable."""
import pytest

from helpers import dev_bf16
from paper_2603_17051_b200 import synth

pytestmark = pytest.mark.gpu


def test_bounded_wait_reports_timeout_and_context_survives():
    import torch
    from paper_2603_17051_b200 import binding as A
    assert A.astro_last_device_status() == 0                  # clean to begin with
    A.astro_selftest_wait_timeout()                           # waits ~1 ms on a barrier nothing completes
    with pytest.raises(A.AstroError) as e:
        A.astro_last_device_status()
    assert e.value.status == 8                                # ASTRO_ERR_TIMEOUT
    assert A.astro_last_device_status() == 0                  # reading cleared the word
    # the context is intact: a normal call still works and leaves the word clean
    q, k, v = (dev_bf16(synth.normal_bf16(77 + i, (1, 130, 2, 64))) for i in range(3))
    o, lse = A.astro_chunk_attn_fwd(None, q, k, v, 0.125)
    torch.cuda.synchronize()
    assert A.astro_last_device_status() == 0
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
