"""Fixed-width bucket indices (LC_OPT_FIXED_WIDTH) and 9-bit promotion (every bucket kept): the "E" and "E+P" stages
of Section 4.3's size breakdown as real streams, against the CPU oracle. Bar: byte-identical streams, bit-identical
recovered fp32 states.
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


def check(lc, oracle, base, cur, nbits, fixed):
    want = oracle.compress(to_np(base), to_np(cur), nbits, fixed=fixed)
    got = lc.compress(base, cur, nbits, fixed=fixed)
    info = lc.stream_info(got)
    assert info.valid == 1 and info.fixed_width == int(fixed) and info.nbits == nbits
    assert to_np(got).tobytes() == want.tobytes()
    out = lc.recover(base, [got])
    assert np.array_equal(to_np(out).view(np.uint32), oracle.recover(to_np(base), [want]).view(np.uint32))
    return got


@pytest.mark.parametrize("n", [0, 1, 5, 4095, 4097, 70001, 1_000_003])
@pytest.mark.parametrize("nbits", [1, 3, 5, 8, 9])
def test_fixed_width_streams(lc, oracle, n, nbits):
    base, cur = make_case(n, 700 + nbits)
    check(lc, oracle, base, cur, nbits, fixed=True)


@pytest.mark.parametrize("fixed", [False, True])
def test_nine_bits_with_more_than_255_buckets(lc, oracle, fixed):
    # magnitudes over 150 binades, both signs: about 300 occupied buckets, symbol ids beyond one byte
    n = 1_500_007
    g = torch.Generator(device=DEV).manual_seed(35)
    mag = torch.exp2(torch.rand(n, generator=g, device=DEV) * 150.0 - 100.0)
    sgn = torch.randint(0, 2, (n,), generator=g, device=DEV) * 2 - 1
    cur = (mag * sgn).to(torch.float32)
    cur[:1000] = 0.0
    base = torch.zeros_like(cur)
    got = check(lc, oracle, base, cur, 9, fixed)
    assert lc.stream_info(got).nsym > 256


def test_paper_example_fixed_width(lc, oracle):
    from conftest import load_golden

    g = load_golden("ten_elements_nbits2.txt")
    cur = torch.from_numpy(g["cur"].copy()).to(DEV)
    base = torch.zeros_like(cur)
    got = check(lc, oracle, base, cur, 9, fixed=True)
    info = lc.stream_info(got)
    assert info.payload_bits == 30 and info.max_len == 3 and info.nsym == 6  # 10 * 3 bits; with 5 * 32: 190 bits


def test_chain_of_mixed_streams_and_fused_update(lc, oracle):
    from paper_2009_13003_b200 import synth

    n = 300_007
    u0 = synth.normal(n, 0.05, DEV, 21)
    u, tracked, streams, streams_np = u0.clone(), u0.clone(), [], []
    for t, (nbits, fixed) in enumerate([(3, False), (9, True), (4, True), (9, False)]):
        u = u + synth.normal(n, 1e-3, DEV, 22 + t)
        s = lc.compress(tracked, u, nbits, fixed=fixed).clone()
        streams.append(s)
        streams_np.append(to_np(s))
        assert streams_np[-1].tobytes() == oracle.compress(to_np(tracked), to_np(u), nbits, fixed=fixed).tobytes()
        tracked = lc.recover(tracked, [s])
    out = lc.recover(u0, streams)
    assert np.array_equal(to_np(out).view(np.uint32), oracle.recover(to_np(u0), streams_np).view(np.uint32))
    assert torch.equal(out.view(torch.int32), tracked.view(torch.int32))
    # the fused call with the fixed-width option: stream and tracked state in one pass
    base, cur = make_case(200_003, 55)
    sbuf, ws = lc.alloc_stream(200_003, 9, DEV), lc.alloc_workspace(200_003, DEV)
    state = torch.empty_like(base)
    lc.compress_opt_async(base, cur, 9, sbuf, ws, lc.OPT_FIXED_WIDTH | lc.OPT_NO_DEVICE_WAIT, tracked_out=state)
    assert lc.last_status(ws) == 0
    want = oracle.compress(to_np(base), to_np(cur), 9, fixed=True)
    assert to_np(sbuf[: want.size]).tobytes() == want.tobytes()
    assert np.array_equal(to_np(state).view(np.uint32), oracle.recover(to_np(base), [want]).view(np.uint32))


def test_three_stages_of_the_size_breakdown(lc):
    # E (every bucket, fixed width) >= E+P (promotion, fixed width) >= E+P+H (Huffman) on a concentrated delta
    from paper_2009_13003_b200 import synth

    n = 2_000_003
    base = synth.normal(n, 0.02, DEV, 3)
    cur = base + synth.lognormal_signed(n, 1e-4, 1.5, DEV, 4)
    e = lc.compress(base, cur, 9, fixed=True).numel()
    ep = lc.compress(base, cur, 3, fixed=True).numel()
    eph = lc.compress(base, cur, 3).numel()
    assert e > ep > eph
    assert eph < 0.10 * 4 * n  # Section 4.3: below 10 % of the full checkpoint with 3-bit promotion
