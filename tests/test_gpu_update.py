"""Parity of lc_compress_update (compress + tracked-state update in one call, Algorithm 1 steps 4-7) with the
CPU oracle: the stream must be byte-identical to the oracle's, and the tracked state bit-identical both to the
oracle's recovery of that stream and to Algorithm 1 step 7 computed directly (no bitstream involved).
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


def check_update(lc, oracle, base, cur, nbits, inplace):
    n = base.numel()
    bh, ch = to_np(base).copy(), to_np(cur).copy()
    cap, wsb, pad = lc.stream_bound(n, nbits), lc.workspace_bytes(n), 256
    sbuf = torch.full((cap + pad,), 0xA5, dtype=torch.uint8, device=DEV)
    wbuf = torch.full((wsb + pad,), 0x5A, dtype=torch.uint8, device=DEV)
    # a canary after the tracked state too (n is often ragged)
    tbuf = torch.full((n + 64,), float("nan"), dtype=torch.float32, device=DEV)
    if inplace:
        tbuf[:n] = base
        src = tbuf[:n]
    else:
        src = base
    lc.compress_update_async(src, cur, nbits, sbuf[:cap], tbuf[:n], wbuf[:wsb])
    assert lc.last_status(wbuf[:wsb]) == 0
    assert bool((sbuf[cap:] == 0xA5).all()) and bool((wbuf[wsb:] == 0x5A).all()), "canary overwritten"
    assert bool(torch.isnan(tbuf[n:]).all()), "wrote past the tracked state"
    info = lc.stream_info(sbuf)
    got = to_np(sbuf[: info.total_bytes])
    want = oracle.compress(bh, ch, nbits)
    assert got.tobytes() == want.tobytes(), "stream differs from the oracle"
    tracked = to_np(tbuf[:n]).view(np.uint32)
    assert np.array_equal(tracked, oracle.recover(bh, [want]).view(np.uint32)), "tracked state != recover(stream)"
    assert np.array_equal(tracked, oracle.apply_quantized(bh, ch, nbits).view(np.uint32)), "tracked state != step 7"
    if not inplace:
        assert np.array_equal(to_np(base).view(np.uint32), bh.view(np.uint32)), "base was modified"
    assert np.array_equal(to_np(cur).view(np.uint32), ch.view(np.uint32)), "cur was modified"
    return got


@pytest.mark.parametrize("n", [1, 5, 127, 4095, 4096, 4097, 32768, 61_706, 300_007, 1_000_003])
@pytest.mark.parametrize("inplace", [False, True])
def test_sizes_and_ragged_tails(lc, oracle, n, inplace):
    base, cur = make_case(n, 100 + n % 97)
    check_update(lc, oracle, base, cur, 1 + n % 8, inplace)


@pytest.mark.parametrize("dist", ["gauss", "lognormal", "one_exp", "one_exp_2sign", "zero"])
@pytest.mark.parametrize("nbits", [2, 5, 8])
def test_distributions(lc, oracle, dist, nbits):
    base, cur = make_case(500_000 + 13, 7, dist=dist)
    check_update(lc, oracle, base, cur, nbits, inplace=(nbits == 5))


@pytest.mark.parametrize("inplace", [False, True])
def test_large_deltas_recompute_keys_from_base(lc, oracle, inplace):
    # exponent fields >= 128: the encode pass reads base again for its keys, also when base is being overwritten
    from paper_2009_13003_b200 import synth

    n = 300_000 + 77
    base = synth.normal(n, 1.0, DEV, 31)
    cur = base + synth.normal(n, 40.0, DEV, 32)
    check_update(lc, oracle, base, cur, 5, inplace)


@pytest.mark.parametrize("inplace", [False, True])
def test_long_codes_and_oversized_chunks(lc, oracle, inplace):
    base, cur = _fibonacci_case(35, True)
    got = check_update(lc, oracle, base, cur, 6, inplace)
    assert got[20] == 34


def test_chain_with_in_place_updates_matches_recovery(lc, oracle):
    # Algorithm 1 as a loop: the tracked state is advanced in place by every compress, and recovering the chain
    # from the first state reproduces it bit for bit.
    from paper_2009_13003_b200 import synth

    n, nbits = 700_001, 4
    u0 = synth.normal(n, 0.02, DEV, 41)
    tracked, u, streams = u0.clone(), u0.clone(), []
    ws = lc.alloc_workspace(n, DEV)
    for t in range(4):
        u = u + synth.lognormal_signed(n, 1e-4, 1.5, DEV, 42 + t)
        s, _ = lc.compress_update(tracked, u, nbits, tracked_out=tracked, workspace=ws)
        streams.append(s.clone())
    out = lc.recover(u0, streams)
    assert torch.equal(out.view(torch.int32), tracked.view(torch.int32))
    want = oracle.recover(to_np(u0), [to_np(s) for s in streams])
    assert np.array_equal(to_np(tracked).view(np.uint32), want.view(np.uint32))


def test_empty_vector_and_argument_errors(lc):
    L = lc.lib()
    e = torch.empty(0, dtype=torch.float32, device=DEV)
    s, t = lc.compress_update(e, e, 3, tracked_out=e)
    assert lc.stream_info(s).n == 0 and t.numel() == 0
    base, cur = make_case(10_000, 3)
    ws, st = lc.alloc_workspace(10_000, DEV), lc.alloc_stream(10_000, 4, DEV)
    cs = lc._cs(base.device)
    args = lambda out: (base.data_ptr(), cur.data_ptr(), 10_000, 4, st.data_ptr(), st.numel(), out, ws.data_ptr(),
                        ws.numel(), cs)
    assert L.lc_compress_update(*args(None)) == lc.ERR_ARG  # no output
    assert L.lc_compress_update(*args(cur.data_ptr())) == lc.ERR_ARG  # output on top of cur
    assert L.lc_compress_update(*args(base.data_ptr() + 4)) == lc.ERR_ARG  # misaligned


def test_nonfinite_delta_leaves_base_untouched(lc):
    base, cur = make_case(100_000, 2)
    cur[77_777] = float("inf")
    keep = base.clone()
    with pytest.raises(lc.LCError) as e:
        lc.compress_update(base, cur, 4, tracked_out=base)
    assert e.value.code == lc.ERR_NONFINITE
    assert torch.equal(base.view(torch.int32), keep.view(torch.int32))


def test_config_xfmr1p3b_full_size_in_place(lc, oracle):
    """The benchmark's workload at full size (1,315,575,808 elements, nbits 5), tracked state advanced in place.

    The stream must equal lc_compress's byte for byte (which test_gpu_parity checks against the oracle at this
    size); the tracked state is compared in full with Algorithm 1 step 7 computed directly on the CPU.
    """
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS["xfmr1p3b"]
    n, nbits = cfg.n, cfg.nbits
    u0 = synth.base_state(cfg, DEV)
    u = u0 + synth.snapshot_delta(cfg, 1, DEV)
    ws = lc.alloc_workspace(n, DEV)
    ref = lc.compress(u0, u, nbits, workspace=ws).clone()
    u0_h, u_h = to_np(u0), to_np(u)
    s, tracked = lc.compress_update(u0, u, nbits, tracked_out=u0, workspace=ws)
    assert tracked.data_ptr() == u0.data_ptr()
    assert torch.equal(s, ref), "stream differs from lc_compress's"
    want = oracle.apply_quantized(u0_h, u_h, nbits)
    assert np.array_equal(to_np(tracked).view(np.uint32), want.view(np.uint32))
