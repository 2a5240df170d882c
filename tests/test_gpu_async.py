"""lc_compress_async: the compress pass split over two CUDA streams (Section 3.2, asynchronous execution). The
stream must be the oracle's, byte for byte, although the model state is overwritten as soon as the statistics pass
has read it.
"""
import numpy as np
import pytest
import torch

from test_gpu_parity import DEV, make_case, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding

    binding.lib()
    return binding


@pytest.mark.parametrize("n,nbits", [(0, 3), (5, 2), (4097, 4), (300_007, 5), (5_000_011, 3)])
def test_two_stream_compress_releases_the_state_early(lc, oracle, n, nbits):
    base, cur = make_case(n, 500 + nbits)
    want = oracle.compress(to_np(base), to_np(cur), nbits)
    state, side = torch.cuda.Stream(DEV), torch.cuda.Stream(DEV)
    ev = torch.cuda.Event()
    sbuf = lc.alloc_stream(n, nbits, DEV)
    ws = lc.alloc_workspace(n, DEV)
    torch.cuda.synchronize()
    lc.compress_two_streams(base, cur, nbits, sbuf, ws, state, side, ev)
    with torch.cuda.stream(state):  # the "next training iteration": overwrites both vectors at once
        cur.fill_(123.0)
        base.fill_(-7.0)
    side.synchronize()
    state.synchronize()
    assert lc.last_status(ws) == 0
    assert to_np(sbuf[: want.size]).tobytes() == want.tobytes()
    assert lc.stream_info(sbuf).total_bytes == want.size


def test_two_stream_compress_rejects_what_it_cannot_do(lc):
    from paper_2009_13003_b200 import synth

    n = 200_000
    base = synth.normal(n, 1.0, DEV, 31)
    cur = base + synth.normal(n, 40.0, DEV, 32)  # deltas of magnitude 2 and more
    state, side = torch.cuda.Stream(DEV), torch.cuda.Stream(DEV)
    ev = torch.cuda.Event()
    sbuf, ws = lc.alloc_stream(n, 5, DEV), lc.alloc_workspace(n, DEV)
    torch.cuda.synchronize()
    lc.compress_two_streams(base, cur, 5, sbuf, ws, state, side, ev)
    torch.cuda.synchronize()
    assert lc.last_status(ws) == lc.ERR_RANGE
    assert lc.stream_info(sbuf).valid == 0
    with pytest.raises(lc.LCError) as e:
        lc.compress_two_streams(base, cur, 5, sbuf, ws, state, state, ev)  # one stream for both roles
    assert e.value.code == lc.ERR_ARG
    rc = lc.lib().lc_compress_async(base.data_ptr(), cur.data_ptr(), n, 5, sbuf.data_ptr(), sbuf.numel(), ws.data_ptr(),
                                    ws.numel(), state.cuda_stream, side.cuda_stream, None)
    assert rc == lc.ERR_ARG
    lc.compress_async(base, cur, 5, sbuf, ws)  # lc_compress handles the same vector
    assert lc.last_status(ws) == 0
