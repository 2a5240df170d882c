"""Parity of lc_merge (Section 3.2, checkpoint merging: the super-step stream of k streams) with the CPU oracle.

Bar: the merged stream is byte-identical to the oracle's, the recovered state left in `scratch` and the state
recovered from the merged stream are bit-identical fp32.
"""
import numpy as np
import pytest
import torch

from test_gpu_parity import DEV, ORACLE_THREADS, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding

    binding.lib()
    return binding


def make_chain(lc, n, k, nbits, seed, scale=1e-3):
    from paper_2009_13003_b200 import synth

    u0 = synth.normal(n, 0.05, DEV, seed)
    u, tracked, streams = u0.clone(), u0.clone(), []
    for t in range(k):
        u = u + synth.normal(n, scale, DEV, seed + 1 + t)
        s = lc.compress(tracked, u, nbits).clone()
        streams.append(s)
        tracked = lc.recover(tracked, [s])
    return u0, streams, tracked


@pytest.mark.parametrize("n,k", [(1, 1), (4097, 2), (70001, 3), (300_007, 1), (300_007, 4), (300_007, 5), (300_007, 8),
                                 (1_000_003, 4)])
def test_merge_matches_the_oracle(lc, oracle, n, k):
    nbits_in, nbits_out = 3, 1 + (n + k) % 8
    u0, streams, tracked = make_chain(lc, n, k, nbits_in, 40 + k)
    scratch = torch.full((n + 16,), float("nan"), dtype=torch.float32, device=DEV)
    got = to_np(lc.merge(u0, streams, nbits_out, scratch=scratch[:n]))
    assert bool(torch.isnan(scratch[n:]).all()), "wrote past the scratch vector"
    assert torch.equal(scratch[:n].view(torch.int32), tracked.view(torch.int32)), "scratch != state of the k streams"
    want = oracle.merge(to_np(u0), [to_np(s) for s in streams], nbits_out)
    assert got.tobytes() == want.tobytes()
    back = lc.recover(u0, [torch.from_numpy(got).to(DEV)])
    assert np.array_equal(to_np(back).view(np.uint32), oracle.recover(to_np(u0), [want]).view(np.uint32))


def test_merge_of_one_stream_over_a_zero_base_is_that_stream(lc):
    from paper_2009_13003_b200 import synth

    n = 500_009
    base = torch.zeros(n, dtype=torch.float32, device=DEV)
    cur = synth.laplace(n, 1e-3, DEV, 91)
    s = lc.compress(base, cur, 4).clone()
    assert torch.equal(lc.merge(base, [s], 4), s)


def test_merge_reports_a_rejected_stream_and_bad_arguments(lc):
    n = 100_000
    u0, streams, _ = make_chain(lc, n, 2, 3, 60)
    bad = streams[1].clone()
    bad[0] = ord("X")
    ws = lc.alloc_workspace(n, DEV)
    out = lc.alloc_stream(n, 4, DEV)
    scratch = torch.empty(n, dtype=torch.float32, device=DEV)
    lc.merge_async(u0, [streams[0], bad], 4, out, scratch, ws)
    assert lc.last_status(ws) == lc.ERR_FORMAT
    assert lc.stream_info(out).valid == 0  # no usable stream is left behind
    lc.merge_async(u0[: n - 1].contiguous(), streams, 4, out, scratch[: n - 1], ws)
    assert lc.last_status(ws) == lc.ERR_MISMATCH
    lc.merge_async(u0, streams, 4, out, scratch, ws)  # and the workspace is fine afterwards
    assert lc.last_status(ws) == 0
    L = lc.lib()
    import ctypes as C

    ptrs = (C.c_void_p * 2)(*[s.data_ptr() for s in streams])
    sizes = (C.c_uint64 * 2)(*[s.numel() for s in streams])
    args = lambda nbits=4, scr=scratch.data_ptr(), cap=out.numel(): (u0.data_ptr(), ptrs, sizes, 2, n, nbits, out.data_ptr(), cap,
                                                                    scr, ws.data_ptr(), ws.numel(), None)
    assert L.lc_merge(*args(nbits=10)) == lc.ERR_ARG
    assert L.lc_merge(*args(scr=None)) == lc.ERR_ARG
    assert L.lc_merge(*args(scr=u0.data_ptr())) == lc.ERR_ARG
    assert L.lc_merge(*args(cap=100)) == lc.ERR_CAPACITY


def test_merge_config_xfmr1p3b_full_size(lc, oracle):
    """The benchmark's chain of 4 merged into one stream at full size, against the oracle on all host cores."""
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS["xfmr1p3b"]
    n, nbits = cfg.n, cfg.nbits
    u0 = synth.base_state(cfg, DEV)
    tracked, u = u0.clone(), u0.clone()
    ws = lc.alloc_workspace(n, DEV)
    streams = []
    for t in range(1, cfg.chain + 1):
        u += synth.snapshot_delta(cfg, t, DEV)
        streams.append(lc.compress(tracked, u, nbits, workspace=ws).clone())
        lc.recover(tracked, [streams[-1]], out=tracked, workspace=ws)
    del u
    scratch = torch.empty_like(u0)
    got = lc.merge(u0, streams, nbits, scratch=scratch, workspace=ws)
    assert torch.equal(scratch.view(torch.int32), tracked.view(torch.int32))
    want = oracle.compress(to_np(u0), to_np(tracked), nbits, threads=ORACLE_THREADS)  # = the oracle's merge, pinned on CPU
    assert got.numel() == want.size
    g = to_np(got)
    for lo in range(0, want.size, 1 << 28):
        assert g[lo: lo + (1 << 28)].tobytes() == want[lo: lo + (1 << 28)].tobytes()
