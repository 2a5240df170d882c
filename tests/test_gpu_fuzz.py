"""Seeded random cases through every compress variant and chained recovery, against the CPU oracle: sizes from 0 to
a few hundred thousand (ragged tails, single chunks), nbits 1...9, deltas that span subnormals to magnitudes beyond
2 (exponent fields the one-byte key plane cannot hold), sparse and constant vectors. Bar: byte-identical streams,
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


def random_case(rng, n):
    """base and a list of successive states; the kind of delta is drawn per case."""
    g = torch.Generator(device="cpu").manual_seed(int(rng.integers(1 << 31)))
    base = (torch.randn(n, generator=g) * float(10.0 ** rng.uniform(-3, 1))).float()
    kind = rng.choice(["normal", "wide", "sparse", "tiny", "const", "two_scales"])
    steps = int(rng.integers(1, 9))
    states, x = [], base
    for _ in range(steps):
        if kind == "normal":
            d = torch.randn(n, generator=g) * float(10.0 ** rng.uniform(-6, -1))
        elif kind == "wide":  # magnitudes over 60 binades, some beyond 2
            d = torch.exp2(torch.randint(-40, 20, (n,), generator=g).float()) * (1 + torch.rand(n, generator=g))
            d = d * torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)
        elif kind == "sparse":
            d = torch.randn(n, generator=g) * 1e-3 * (torch.rand(n, generator=g) < 0.05)
        elif kind == "tiny":  # down into the subnormals
            d = torch.exp2(torch.randint(-149, -120, (n,), generator=g).float())
        elif kind == "const":
            d = torch.full((n,), float(rng.uniform(-1e-2, 1e-2)))
        else:
            d = torch.randn(n, generator=g) * torch.where(torch.arange(n) < n // 2, 1e-5, 1e-1)
        x = (x + d.float()).float()
        states.append(x)
    return base.to(DEV), [s.to(DEV) for s in states], kind


@pytest.mark.parametrize("seed", range(64))
def test_random_cases(lc, oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.choice([0, 1, 3, 4, 127, 4095, 4096, 4097, int(rng.integers(5, 20_000)), int(rng.integers(20_000, 400_000))]))
    nbits = int(rng.integers(1, 10))
    base, states, kind = random_case(rng, n)
    tracked = base.clone()
    host = to_np(base).copy()
    cache, ocache = lc.alloc_length_cache(DEV), oracle.new_cache()
    ws = lc.alloc_workspace(n, DEV)
    streams, want_streams = [], []
    for t, cur in enumerate(states):
        cur_h = to_np(cur)
        variant = ["plain", "update", "no_wait", "cached"][int(rng.integers(4))]
        want = oracle.compress_cached(host, cur_h, nbits, ocache) if variant == "cached" else oracle.compress(host, cur_h, nbits)
        sb = lc.alloc_stream(n, nbits, DEV)
        if variant == "plain":
            lc.compress_async(tracked, cur, nbits, sb, ws)
        elif variant == "update":
            lc.compress_update_async(tracked, cur, nbits, sb, tracked, ws)
        elif variant == "no_wait":
            lc.compress_opt_async(tracked, cur, nbits, sb, ws, lc.OPT_NO_DEVICE_WAIT)
        else:
            lc.compress_cached_async(tracked, cur, nbits, sb, ws, cache)
        assert lc.last_status(ws) == 0, (variant, kind)
        size = lc.stream_info(sb).total_bytes
        assert to_np(sb[:size]).tobytes() == want.tobytes(), (t, variant, kind, n, nbits)
        host = oracle.recover(host, [want])
        if variant != "update":
            lc.recover(tracked, [sb[:size]], out=tracked, workspace=ws)
        assert np.array_equal(to_np(tracked).view(np.uint32), host.view(np.uint32)), (t, variant, kind)
        streams.append(sb[:size])
        want_streams.append(want)
        # the other representations of the same snapshot decode to what the oracle says
        if t == 0:
            for mode, ostream in (("fixed", oracle.compress(to_np(base), cur_h, nbits, fixed=True)),
                                  ("mean", oracle.compress_mean(to_np(base), cur_h, nbits))):
                got = lc.compress(base, cur, nbits, fixed=(mode == "fixed"), mean=(mode == "mean"))
                assert to_np(got).tobytes() == ostream.tobytes(), (mode, kind, n, nbits)
                assert np.array_equal(to_np(lc.recover(base, [got])).view(np.uint32),
                                      oracle.recover(to_np(base), [ostream]).view(np.uint32)), (mode, kind)
    # the whole chain from the first base, and its merge
    out = lc.recover(base, streams)
    assert np.array_equal(to_np(out).view(np.uint32), host.view(np.uint32))
    merged = lc.merge(base, streams, nbits)
    assert to_np(merged).tobytes() == oracle.merge(to_np(base), want_streams, nbits).tobytes()
