"""The two ways the encode pass places its chunks (look-back between running CTAs, or a separate scan), the
bounded wait of the first, and run-to-run determinism of the recovery and fused-update calls.

Bar: byte-identical streams (integer work), bit-identical fp32 states.
"""
import numpy as np
import pytest
import torch

from test_gpu_parity import DEV, _fibonacci_case, make_case, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding

    binding.lib()
    return binding


def compress_no_wait(lc, base, cur, nbits, tracked_out=None):
    n = base.numel()
    cap, wsb, pad = lc.stream_bound(n, nbits), lc.workspace_bytes(n), 256
    sbuf = torch.full((cap + pad,), 0xA5, dtype=torch.uint8, device=DEV)
    wbuf = torch.full((wsb + pad,), 0x5A, dtype=torch.uint8, device=DEV)
    lc.compress_opt_async(base, cur, nbits, sbuf[:cap], wbuf[:wsb], lc.OPT_NO_DEVICE_WAIT, tracked_out)
    assert lc.last_status(wbuf[:wsb]) == 0
    assert bool((sbuf[cap:] == 0xA5).all()) and bool((wbuf[wsb:] == 0x5A).all()), "canary overwritten"
    return to_np(sbuf[: lc.stream_info(sbuf).total_bytes])


@pytest.mark.parametrize("n", [0, 1, 4095, 4096, 4097, 8 * 4096 + 1, 70001, 61 * 4096 + 2049, 1_000_003, 5_000_011])
def test_two_pass_scan_writes_the_oracle_stream(lc, oracle, n):
    nbits = 1 + n % 8
    base, cur = make_case(n, 300 + n % 1000)
    got = compress_no_wait(lc, base, cur, nbits)
    assert got.tobytes() == oracle.compress(to_np(base), to_np(cur), nbits).tobytes()


@pytest.mark.parametrize("dist,nbits", [("lognormal", 5), ("gauss", 8), ("one_exp_2sign", 2), ("zero", 4)])
def test_two_pass_scan_distributions_and_tracked_state(lc, oracle, dist, nbits):
    from paper_2009_13003_b200 import synth

    n = (1 << 20) + 4096 * 5 + 3
    base = synth.normal(n, 0.02, DEV, 17)
    if dist.startswith("one_exp"):
        base = torch.zeros_like(base)
    cur = base + synth.sweep_delta(dist, n, DEV, 19 + nbits)
    want = oracle.compress(to_np(base), to_np(cur), nbits)
    tracked = torch.empty_like(base)
    got = compress_no_wait(lc, base, cur, nbits, tracked_out=tracked)
    assert got.tobytes() == want.tobytes()
    assert np.array_equal(to_np(tracked).view(np.uint32), oracle.recover(to_np(base), [want]).view(np.uint32))


def test_two_pass_scan_special_paths(lc, oracle):
    # codes beyond 32 bits with oversized leading chunks, and exponent fields the one-byte key plane cannot hold
    from paper_2009_13003_b200 import synth

    base, cur = _fibonacci_case(35, True)
    assert compress_no_wait(lc, base, cur, 6).tobytes() == oracle.compress(to_np(base), to_np(cur), 6).tobytes()
    n = 300_000 + 77
    base = synth.normal(n, 1.0, DEV, 31)
    cur = base + synth.normal(n, 40.0, DEV, 32)
    assert compress_no_wait(lc, base, cur, 5).tobytes() == oracle.compress(to_np(base), to_np(cur), 5).tobytes()


def test_bounded_wait_runs_out_and_the_next_call_is_fine(lc, oracle):
    """Tile 0 is never coded (the first ticket handed out is 1), so its descriptor never appears: the CTA that needs
    it gives up after a few hundred polls, the others see the abort mark, the call ends with LC_ERR_TIMEOUT. Every
    wait is bounded, so nothing can hang. A normal call on the same workspace then succeeds."""
    n, nbits = 64 * 4096 + 100, 4  # nine tiles of eight chunks
    base, cur = make_case(n, 77)
    ws = lc.alloc_workspace(n, DEV)
    sbuf = lc.alloc_stream(n, nbits, DEV)
    for spin_limit in (0, 300):
        lc.debug_compress_wait(base, cur, nbits, sbuf, ws, spin_limit, 1)
        assert lc.last_status(ws) == lc.ERR_TIMEOUT
    # with the first ticket at 0 the same entry point is lc_compress, also with a small limit that is never reached
    # on a vector of one tile
    small = 5 * 4096
    lc.debug_compress_wait(base[:small], cur[:small], nbits, sbuf, ws, 0, 0)
    assert lc.last_status(ws) == 0
    want = oracle.compress(to_np(base[:small]), to_np(cur[:small]), nbits)
    assert to_np(sbuf[: want.size]).tobytes() == want.tobytes()
    lc.compress_async(base, cur, nbits, sbuf, ws)
    assert lc.last_status(ws) == 0
    want = oracle.compress(to_np(base), to_np(cur), nbits)
    assert to_np(sbuf[: want.size]).tobytes() == want.tobytes()


def test_recover_and_fused_update_are_deterministic(lc):
    n = 5_000_011
    base, cur = make_case(n, 5)
    s, t0 = lc.compress_update(base, cur, 5)
    s0 = s.clone()
    for _ in range(3):
        s1, t1 = lc.compress_update(base, cur, 5)
        assert torch.equal(s0, s1) and torch.equal(t0.view(torch.int32), t1.view(torch.int32))
    for k in (1, 2, 4):
        r0 = lc.recover(base, [s0] * k)
        for _ in range(3):
            assert torch.equal(r0.view(torch.int32), lc.recover(base, [s0] * k).view(torch.int32))
    x = base.clone()
    lc.recover(x, [s0, s0], out=x)  # in place
    assert torch.equal(x.view(torch.int32), lc.recover(base, [s0, s0]).view(torch.int32))
