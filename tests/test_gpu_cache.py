"""Huffman code table caching (Section 3.2): lc_compress_cached against the CPU oracle over a sequence of snapshots
that share one length cache. Bar: after every snapshot the stream and the whole cache are byte-identical to the
oracle's, and the recovered fp32 state is bit-identical to the plain stream's.
"""
import numpy as np
import pytest
import torch

from test_gpu_parity import DEV, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding

    binding.lib()
    return binding


def snapshots(n, seed):
    """Deltas whose length lists differ: hits that are not optimal, a row the size bound rejects, rows of other
    symbol counts, fewer than two used symbols."""
    from paper_2009_13003_b200 import synth

    base = synth.normal(n, 0.02, DEV, seed)
    deltas = [
        synth.normal(n, 1e-3, DEV, seed + 1),                    # flat length list: fills the row
        synth.laplace(n, 1e-3, DEV, seed + 2),                   # steep distribution coded with the flat list: a hit
        synth.laplace(n, 3e-4, DEV, seed + 3),                   # another hit
        synth.lognormal_signed(n, 1e-4, 1.5, DEV, seed + 4),     # wide: more buckets, maybe another row
        synth.one_exponent(n, -13, DEV, seed + 5, two_sign=True),  # two used symbols
        torch.zeros(n, dtype=torch.float32, device=DEV),         # one used symbol: no code, cache untouched
        synth.laplace(n, 1e-3, DEV, seed + 6),
        synth.normal(n, 1e-3, DEV, seed + 7),                    # the steep list on the flat distribution
    ]
    return base, [base + d for d in deltas]


@pytest.mark.parametrize("n,nbits", [(3 * 4096 + 500, 3), (200_003, 5), (1_000_003, 9), (50_000, 1)])
def test_cached_sequence_matches_the_oracle(lc, oracle, n, nbits):
    base, curs = snapshots(n, 40 + nbits)
    cache = lc.alloc_length_cache(DEV)
    want_cache = oracle.new_cache()
    hits = 0
    for cur in curs:
        want = oracle.compress_cached(to_np(base), to_np(cur), nbits, want_cache)
        got = lc.compress_cached(base, cur, nbits, cache)
        assert to_np(got).tobytes() == want.tobytes()
        assert to_np(cache).tobytes() == want_cache.tobytes()
        info = lc.stream_info(got)
        assert info.valid == 1 and info.cached_lengths == (int(want[7]) >> 2)
        hits += info.cached_lengths
        plain = lc.compress(base, cur, nbits)
        assert lc.stream_info(plain).payload_bits <= info.payload_bits <= n * nbits
        assert torch.equal(lc.recover(base, [got]), lc.recover(base, [plain]))
    assert hits >= 2  # the sequence is built to reuse rows


def test_cached_with_tracked_state_and_arguments(lc, oracle):
    n, nbits = 70_001, 4
    base, curs = snapshots(n, 77)
    cache = lc.alloc_length_cache(DEV)
    want_cache = oracle.new_cache()
    tracked = base.clone()
    host = to_np(base).copy()
    for cur in curs[:4]:
        # a chain: every snapshot is coded against the tracked state, which the same call moves on
        want = oracle.compress_cached(host, to_np(cur), nbits, want_cache)
        host = oracle.recover(host, [want])
        got = lc.compress_cached(tracked, cur, nbits, cache, tracked_out=tracked)
        assert to_np(got).tobytes() == want.tobytes()
        assert np.array_equal(to_np(tracked).view(np.uint32), host.view(np.uint32))
    ws = lc.alloc_workspace(n, DEV)
    sb = lc.alloc_stream(n, nbits, DEV)
    L = lc.lib()
    args = (base.data_ptr(), curs[0].data_ptr(), n, nbits, sb.data_ptr(), sb.numel(), None, ws.data_ptr(), ws.numel())
    assert L.lc_compress_cached(*args, None, None) == lc.ERR_ARG
    assert L.lc_compress_cached(*args, cache.data_ptr() + 4, None) == lc.ERR_ARG
