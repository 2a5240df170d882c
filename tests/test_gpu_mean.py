"""Mean representatives (LC_OPT_MEAN_REP, format section 1.8) against the CPU oracle. Bar: byte-identical streams
(the representatives are exact integer means, so no tolerance), bit-identical recovered fp32 states.
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


def check(lc, oracle, base, cur, nbits):
    want = oracle.compress_mean(to_np(base), to_np(cur), nbits)
    got = lc.compress(base, cur, nbits, mean=True)
    info = lc.stream_info(got)
    assert info.valid == 1 and info.mean_rep == 1 and info.nbits == nbits
    assert to_np(got).tobytes() == want.tobytes()
    out = lc.recover(base, [got])
    assert np.array_equal(to_np(out).view(np.uint32), oracle.recover(to_np(base), [want]).view(np.uint32))
    return got


@pytest.mark.parametrize("n", [0, 1, 5, 1023, 1025, 4097, 70001, 1_000_003])
@pytest.mark.parametrize("nbits", [1, 3, 5, 9])
def test_mean_streams(lc, oracle, n, nbits):
    base, cur = make_case(n, 900 + nbits)
    check(lc, oracle, base, cur, nbits)


@pytest.mark.parametrize("dist", ["gauss", "lognormal", "one_exp", "one_exp_2sign", "zero"])
def test_mean_streams_by_distribution(lc, oracle, dist):
    base, cur = make_case(300_007, 950, dist=dist)
    check(lc, oracle, base, cur, 4)


def test_mean_with_large_and_tiny_deltas(lc, oracle):
    # exponent fields above 127 (the one-byte key plane does not identify them), subnormal deltas, both signs
    n = 50_000
    g = torch.Generator(device="cpu").manual_seed(5)
    mag = torch.exp2(torch.randint(-140, 100, (n,), generator=g).float()) * (1 + torch.rand(n, generator=g))
    sign = torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)
    cur = (mag * sign).to(DEV)
    base = torch.zeros(n, dtype=torch.float32, device=DEV)
    for nbits in (2, 6, 9):
        check(lc, oracle, base, cur, nbits)


def test_mean_with_tracked_state_and_options(lc, oracle):
    n, nbits = 123_457, 4
    base, cur = make_case(n, 990)
    want = oracle.compress_mean(to_np(base), to_np(cur), nbits)
    ws, sb = lc.alloc_workspace(n, DEV), lc.alloc_stream(n, nbits, DEV)
    tracked = torch.empty_like(base)
    L = lc.lib()
    args = (base.data_ptr(), cur.data_ptr(), n, nbits, sb.data_ptr(), sb.numel(), tracked.data_ptr(), ws.data_ptr(), ws.numel())
    for options in (lc.OPT_MEAN_REP, lc.OPT_MEAN_REP | lc.OPT_NO_DEVICE_WAIT):
        sb.zero_()
        assert L.lc_compress_opt(*args, options, None) == 0
        assert lc.last_status(ws) == 0
        assert to_np(sb)[: want.size].tobytes() == want.tobytes()
        assert np.array_equal(to_np(tracked).view(np.uint32), oracle.recover(to_np(base), [want]).view(np.uint32))
    assert L.lc_compress_opt(*args, lc.OPT_MEAN_REP | lc.OPT_FIXED_WIDTH, None) == lc.ERR_ARG
    # the default pass after the variant: the plain stream again
    plain = lc.compress(base, cur, nbits, workspace=ws)
    assert to_np(plain).tobytes() == oracle.compress(to_np(base), to_np(cur), nbits).tobytes()
