"""lc_compress_noalloc against lc_compress and the CPU oracle (collected last on purpose: a failure here must not
hide others).

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


def test_noalloc_matches_workspace_entry_point_twice(oracle):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding as lc
    from paper_2009_13003_b200 import synth

    # the start-up call a caller makes before its pool takes the device: n = 0 resolves the scratch array (and
    # loads the part of the library that holds it) and writes a header-only stream
    empty = torch.empty(0, dtype=torch.float32, device=DEV)
    buf0 = torch.empty(lc.stream_bound(0, 3), dtype=torch.uint8, device=DEV)
    got0 = lc.compress_noalloc(empty, empty, 3, buf0).cpu().numpy()
    assert got0.tobytes() == oracle.compress(np.zeros(0, np.float32), np.zeros(0, np.float32), 3).tobytes()

    cases = [(1_000_003, 5, 71), (262_144 + 77, 3, 72)]  # second call: smaller n, other nbits, same array
    for n, nbits, seed in cases:
        base = synth.normal(n, 0.02, DEV, seed)
        cur = base + synth.lognormal_signed(n, 1e-4, 1.5, DEV, seed + 100)
        want = lc.compress(base, cur, nbits).cpu().numpy()
        buf = torch.full((lc.stream_bound(n, nbits) + 64,), 0xA5, dtype=torch.uint8, device=DEV)
        got = lc.compress_noalloc(base, cur, nbits, buf[: lc.stream_bound(n, nbits)]).cpu().numpy()
        assert got.tobytes() == want.tobytes()  # integer / byte work: bit-exact
        assert got.tobytes() == oracle.compress(base.cpu().numpy(), cur.cpu().numpy(), nbits).tobytes()
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
    rc = lc.lib().lc_compress_noalloc(x.data_ptr(), x.data_ptr(), 16, 10, buf.data_ptr(), buf.numel(), None)
    assert rc == lc.ERR_ARG
