"""One process, two devices: the launch parameters the library caches (SM count, CTAs per SM, raised shared-memory
limits) are kept per device, so a call on a second GPU must work after calls on the first. Skipped where fewer than
two devices are visible.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_calls_on_device_0_then_device_1(oracle):
    if not torch.cuda.is_available() or torch.cuda.device_count() < 2:
        pytest.skip("needs two CUDA devices")
    from paper_2009_13003_b200 import binding as lc, synth

    n, nbits = 300_007, 4
    for dev in ("cuda:0", "cuda:1", "cuda:0"):
        with torch.cuda.device(dev):
            base = synth.normal(n, 0.02, dev, 1)
            cur = base + synth.laplace(n, 1e-3, dev, 2)
            s = lc.compress(base, cur, nbits)
            want = oracle.compress(base.cpu().numpy(), cur.cpu().numpy(), nbits)
            assert s.cpu().numpy().tobytes() == want.tobytes()
            out = lc.recover(base, [s, s])
            assert np.array_equal(out.cpu().numpy().view(np.uint32),
                                  oracle.recover(base.cpu().numpy(), [want, want]).view(np.uint32))
