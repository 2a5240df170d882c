"""Per-layer granularity (lc_compress_segments / lc_recover_segments): every segment's stream must be the oracle's
stream of that slice, and the recovered vector the oracle's recovery segment by segment. Bar: byte-identical streams,
bit-identical fp32 states.
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


def layered_case(sizes, seed, chain):
    """A state of len(sizes) layers whose updates differ in scale by layer (two decades), `chain` snapshots."""
    from paper_2009_13003_b200 import synth

    n = sum(sizes)
    base = synth.normal(n, 0.05, DEV, seed)
    begin = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    scale = torch.empty(n, dtype=torch.float32, device=DEV)
    for i, (a, b) in enumerate(zip(begin[:-1], begin[1:])):
        scale[a:b] = 1e-4 * 100.0 ** (((i * 7) % len(sizes)) / max(1, len(sizes) - 1))
    curs, x = [], base
    for t in range(chain):
        x = x + synth.normal(n, 1.0, DEV, seed + 1 + t) * scale
        curs.append(x)
    return base, curs, [int(v) for v in begin]


@pytest.mark.parametrize("sizes,nbits", [
    ([9408, 64, 64, 36864, 64, 0, 4, 70000, 1000], 4),
    ([4096 * 3, 4096, 8], 2),
    ([1_000_000, 12, 300_000], 5),
])
def test_segments_match_the_oracle_slice_by_slice(lc, oracle, sizes, nbits):
    base, curs, begin = layered_case(sizes, 300 + nbits, chain=3)
    offsets, total = lc.segments_layout(begin, nbits)
    assert offsets[0] == 0 and offsets[-1] == total and all(o % 256 == 0 for o in offsets)
    tracked = base.clone()
    host = to_np(base).copy()
    bufs = []
    for cur in curs:
        want = [oracle.compress(host[a:b], to_np(cur)[a:b], nbits) for a, b in zip(begin[:-1], begin[1:])]
        streams, off = lc.compress_segments(tracked, cur, begin, nbits, tracked_out=tracked)
        assert off == offsets
        got = to_np(streams)
        for i, w in enumerate(want):
            assert got[off[i]: off[i] + w.size].tobytes() == w.tobytes(), "segment %d" % i
            assert w.size <= off[i + 1] - off[i]
        for (a, b), w in zip(zip(begin[:-1], begin[1:]), want):
            host[a:b] = oracle.recover(host[a:b], [w])
        assert np.array_equal(to_np(tracked).view(np.uint32), host.view(np.uint32))
        bufs.append(streams)
    # the chain recovered from the first base, all segments, all snapshots
    out = lc.recover_segments(base, bufs, begin, nbits)
    assert np.array_equal(to_np(out).view(np.uint32), host.view(np.uint32))
    # per-layer tables keep small-scale layers that the table of the flat vector drops entirely
    flat = lc.recover(base, [lc.compress(base, curs[0], nbits)])
    seg1 = lc.recover_segments(base, bufs[:1], begin, nbits)
    err_flat = float((flat - curs[0]).abs().sum())
    err_seg = float((seg1 - curs[0]).abs().sum())
    if len([s for s in sizes if s > 1000]) > 1:
        assert err_seg < err_flat


def test_segments_arguments_and_failures(lc, oracle):
    sizes = [4096, 8192, 4096]
    base, curs, begin = layered_case(sizes, 77, chain=1)
    cur = curs[0].clone()
    nbits = 3
    L = lc.lib()
    import ctypes as C

    def layout(b):
        arr = (C.c_uint64 * len(b))(*b)
        return int(L.lc_segments_layout(arr, len(b) - 1, nbits, None))

    assert layout(begin) > 0
    assert layout([0, 4096, 4098, 16384]) == 0      # a segment that does not start on a 16-byte boundary
    assert layout([4, 4096, 8192, 16384]) == 0      # does not start at 0
    assert layout([0, 8192, 4096, 16384]) == 0      # decreasing
    offsets, total = lc.segments_layout(begin, nbits)
    ws = lc.alloc_workspace(max(sizes), DEV)
    small = torch.empty(total - 256, dtype=torch.uint8, device=DEV)
    with pytest.raises(lc.LCError) as e:
        lc.compress_segments_async(base, cur, begin, nbits, small, ws)
    assert e.value.code == lc.ERR_CAPACITY
    # a non-finite delta in the middle segment: the status word keeps that failure, the first segment's stream is
    # complete, the failed and the following segment have no valid stream
    cur[5000] = float("inf")
    streams = torch.zeros(total, dtype=torch.uint8, device=DEV)
    lc.compress_segments_async(base, cur, begin, nbits, streams, ws)
    assert lc.last_status(ws) == lc.ERR_NONFINITE
    first = oracle.compress(to_np(base)[:4096], to_np(cur)[:4096], nbits)
    assert to_np(streams)[: first.size].tobytes() == first.tobytes()
    for i in (1, 2):
        assert lc.stream_info(streams[offsets[i]:]).valid == 0
    # and the next call starts clean
    cur[5000] = 0.0
    streams, _ = lc.compress_segments(base, cur, begin, nbits)
    out = lc.recover_segments(base, [streams], begin, nbits)
    want = np.concatenate([oracle.recover(to_np(base)[a:b], [oracle.compress(to_np(base)[a:b], to_np(cur)[a:b], nbits)])
                           for a, b in zip(begin[:-1], begin[1:])])
    assert np.array_equal(to_np(out).view(np.uint32), want.view(np.uint32))
    # a damaged stream in one segment is reported by recover
    bad = streams.clone()
    bad[offsets[1]] = 0
    with pytest.raises(lc.LCError) as e:
        lc.recover_segments(base, [bad], begin, nbits)
    assert e.value.code == lc.ERR_FORMAT
