"""lc_compress_noalloc against lc_compress (collected last on purpose: a failure here must not hide others).

The entry point serves callers that cannot allocate device memory when they take a snapshot (their
pool owns the device, or allocation is forbidden where they run); its scratch is an array inside the
library. It has to produce exactly the stream lc_compress produces, also on a second call that finds
the first call's leftovers in that shared array.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def test_noalloc_matches_workspace_entry_point_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding as lc
    from paper_2009_13003_b200 import synth

    cases = [(1_000_003, 5, 71), (262_144 + 77, 3, 72)]  # second call: smaller n, other nbits, same array
    for n, nbits, seed in cases:
        base = synth.normal(n, 0.02, DEV, seed)
        cur = base + synth.lognormal_signed(n, 1e-4, 1.5, DEV, seed + 100)
        want = lc.compress(base, cur, nbits).cpu().numpy()
        buf = torch.full((lc.stream_bound(n, nbits) + 64,), 0xA5, dtype=torch.uint8, device=DEV)
        got = lc.compress_noalloc(base, cur, nbits, buf[: lc.stream_bound(n, nbits)]).cpu().numpy()
        assert got.tobytes() == want.tobytes()  # integer / byte work: bit-exact
        assert bool((buf[lc.stream_bound(n, nbits):] == 0xA5).all())
        # and the stream decodes to the same state
        a = lc.recover(base, [torch.from_numpy(got).to(DEV)])
        b = lc.recover(base, [torch.from_numpy(want).to(DEV)])
        assert torch.equal(a, b)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding as lc

    n = lc.NOALLOC_MAX_N + 1
    x = torch.zeros(n, dtype=torch.float32, device=DEV)
    buf = torch.empty(lc.stream_bound(n, 4), dtype=torch.uint8, device=DEV)
    rc = lc.lib().lc_compress_noalloc(x.data_ptr(), x.data_ptr(), n, 4, buf.data_ptr(), buf.numel(), None)
    assert rc == lc.ERR_CAPACITY
    rc = lc.lib().lc_compress_noalloc(x.data_ptr(), x.data_ptr(), 16, 9, buf.data_ptr(), buf.numel(), None)
    assert rc == lc.ERR_ARG
