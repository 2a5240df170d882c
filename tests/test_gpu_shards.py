"""A vector split into shards that are coded separately with the table of the whole vector (lc_shard_stats, the
exchange of the 512 bucket statistics, lc_shard_encode), against the CPU oracle. One GPU stands in for all devices:
the shards are processed one after the other and their statistics combined with the function an all-reduce computes.
Bar: byte-identical streams, bit-identical recovered fp32 states.
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


def heterogeneous_case(n, seed):
    from paper_2009_13003_b200 import synth

    base = synth.normal(n, 0.02, DEV, seed)
    d = synth.laplace(n, 1e-3, DEV, seed + 1)
    d[: n // 3] *= 40.0  # the parts differ in scale: the whole vector's table is not any part's own
    return base, base + d


@pytest.mark.parametrize("n,cuts,nbits", [
    (5 * 4096 + 321, [0, 2 * 4096, 3 * 4096], 3),          # chunk-aligned cuts
    (1_000_003, [0, 250_000, 250_004, 700_008], 5),        # cuts inside chunks (multiples of 4 elements), a tiny shard
    (300_007, [0], 4),                                     # one shard: the whole vector
    (40_000, [0, 20_000, 20_000], 2),                      # an empty shard
])
def test_shards_match_the_oracle(lc, oracle, n, cuts, nbits):
    base, cur = heterogeneous_case(n, 800 + nbits)
    bh, ch = to_np(base), to_np(cur)
    bounds = list(zip(cuts, cuts[1:] + [n]))
    work = [lc.alloc_workspace(hi - lo, DEV) for lo, hi in bounds]
    stats = [lc.shard_stats(base[lo:hi], cur[lo:hi], w) for (lo, hi), w in zip(bounds, work)]
    whole = lc.combine_stats(stats)
    whole_state = oracle.recover(bh, [oracle.compress(bh, ch, nbits)])
    for (lo, hi), w in zip(bounds, work):
        s = lc.shard_encode(base[lo:hi], cur[lo:hi], nbits, whole, w)
        want = oracle.compress_shard(bh, ch, lo, hi, nbits)
        assert to_np(s).tobytes() == want.tobytes(), (lo, hi)
        info = lc.stream_info(s)
        assert info.valid == 1 and info.shard == 1 and info.n == hi - lo
        out = lc.recover(base[lo:hi].contiguous(), [s])
        assert np.array_equal(to_np(out).view(np.uint32), whole_state[lo:hi].view(np.uint32))
    if len(bounds) == 1:
        plain = to_np(lc.compress(base, cur, nbits)).copy()
        plain[7] |= 2
        assert to_np(lc.shard_encode(base, cur, nbits, whole, work[0])).tobytes() == plain.tobytes()


def test_a_nonfinite_delta_in_one_shard_stops_every_shard(lc):
    n = 200_000
    base, cur = heterogeneous_case(n, 900)
    cur[150_000] = float("inf")
    halves = [(0, 100_000), (100_000, n)]
    work = [lc.alloc_workspace(hi - lo, DEV) for lo, hi in halves]
    whole = lc.combine_stats([lc.shard_stats(base[lo:hi], cur[lo:hi], w) for (lo, hi), w in zip(halves, work)])
    for (lo, hi), w in zip(halves, work):
        with pytest.raises(lc.LCError) as e:
            lc.shard_encode(base[lo:hi], cur[lo:hi], 4, whole, w)
        assert e.value.code == lc.ERR_NONFINITE
