"""Parity of the CUDA path (through the C ABI) with the CPU oracle, on the same seeded inputs.

Bar: bit-exact for every integer / byte / index result (bucket statistics, selected keys, symbols,
codebook, whole stream) and bit-exact fp32 for the recovered state (the representative is computed in
integers on the GPU and in double on the CPU, both exact; spec tolerance 1e-6 relative is the
fallback threshold stated in ``REL_TOL`` and checked as well).
"""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

REL_TOL = 1e-6
# host threads for the oracle's chunk-parallel mode (byte-identical to its single-threaded pass, pinned on the CPU)
ORACLE_THREADS = max(1, min(os.cpu_count() or 1, 64))


@pytest.fixture(scope="module")
def lc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2009_13003_b200 import binding

    binding.lib()
    return binding


DEV = "cuda:0"


def to_np(t):
    return t.detach().cpu().numpy()


def gpu_compress(lc, base, cur, nbits, canary=True):
    """Compress with canaries behind the stream and workspace buffers; returns (stream np, workspace)."""
    n = base.numel()
    cap, wsb = lc.stream_bound(n, nbits), lc.workspace_bytes(n)
    pad = 256
    sbuf = torch.full((cap + pad,), 0xA5, dtype=torch.uint8, device=DEV)
    wbuf = torch.full((wsb + pad,), 0x5A, dtype=torch.uint8, device=DEV)
    lc.compress_async(base, cur, nbits, sbuf[:cap], wbuf[:wsb])
    st = lc.last_status(wbuf[:wsb])
    assert bool((sbuf[cap:] == 0xA5).all()) and bool((wbuf[wsb:] == 0x5A).all()), "canary overwritten"
    if st != 0:
        raise lc.LCError(st, "device")
    info = lc.stream_info(sbuf)
    assert info.valid == 1 and info.total_bytes <= cap
    return to_np(sbuf[: info.total_bytes]), wbuf[:wsb]


def assert_stream_parity(lc, oracle, base, cur, nbits):
    bh, ch = to_np(base), to_np(cur)
    got, ws = gpu_compress(lc, base, cur, nbits)
    # stage by stage, so that a failure names the step
    count, mmin, mmax = lc.debug_bins(ws)
    ocount, omin, omax = oracle.bins(bh, ch)
    assert np.array_equal(count, ocount), "histogram"
    assert np.array_equal(mmin, omin) and np.array_equal(mmax, omax), "bucket min/max"
    t = oracle.table(bh, ch, nbits)
    ln, code = lc.debug_codes(ws)
    sym_of_key = np.zeros(512, np.int64)
    sym_of_key[t["key"][1:]] = np.arange(1, len(t["key"]))
    assert np.array_equal(ln, t["len"][sym_of_key].astype(np.uint32)), "code lengths"
    assert np.array_equal(code, t["code"][sym_of_key]), "codes"
    want = oracle.compress(bh, ch, nbits)
    assert got.size == want.size, "stream size"
    nsym = len(t["key"])
    assert got[:64].tobytes() == want[:64].tobytes(), "header"
    assert got[64:64 + 16 * nsym].tobytes() == want[64:64 + 16 * nsym].tobytes(), "symbol table"
    assert got.tobytes() == want.tobytes(), "indices / payload"
    return got, want


def assert_recover_parity(lc, oracle, base, streams_np, inplace=False):
    streams = [torch.from_numpy(s).to(DEV) for s in streams_np]
    want = oracle.recover(to_np(base), streams_np)
    if inplace:
        x = base.clone()
        out = lc.recover(x, streams, out=x)
    else:
        out = lc.recover(base, streams)
    got = to_np(out)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), "recovered state"
    denom = np.maximum(np.abs(want), np.float32(1e-30))
    assert float(np.max(np.abs(got - want) / denom, initial=0.0)) <= REL_TOL
    return got


def make_case(n, seed, scale=1e-3, dist="laplace"):
    from paper_2009_13003_b200 import synth

    base = synth.normal(n, 0.02, DEV, seed)
    d = synth.sweep_delta(dist, n, DEV, seed + 1) if dist != "laplace" else synth.laplace(n, scale, DEV, seed + 1)
    return base, base + d


# ----------------------------------------------------------------------------------------------------


def test_library_identifies_itself(lc):
    assert lc.lib().lc_version() == 100


@pytest.mark.parametrize("name", ["ten_elements_nbits2.txt", "skew16_nbits3.txt"])
def test_golden_streams(lc, name):
    from conftest import load_golden

    g = load_golden(name)
    cur = torch.from_numpy(g["cur"].copy()).to(DEV)
    base = torch.zeros_like(cur)
    got, _ = gpu_compress(lc, base, cur, g["nbits"])
    assert got.tobytes() == g["stream"].tobytes()
    out = lc.recover(base, [torch.from_numpy(g["stream"].copy()).to(DEV)])
    assert to_np(out).view(np.uint32).tolist() == g["recovered"].view(np.uint32).tolist()


SIZES = [0, 1, 3, 4, 5, 127, 128, 129, 1023, 1024, 1025, 4095, 4096, 4097, 3 * 4096 + 77, 8 * 4096,
         8 * 4096 + 1, 70001, 61 * 4096 + 2049, 1_000_003]


@pytest.mark.parametrize("n", SIZES)
def test_sizes_and_ragged_tails(lc, oracle, n):
    nbits = 1 + n % 8
    base, cur = make_case(n, 100 + n % 1000)
    got, _ = assert_stream_parity(lc, oracle, base, cur, nbits)
    assert_recover_parity(lc, oracle, base, [got])


@pytest.mark.parametrize("nbits", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("dist", ["gauss", "laplace", "lognormal", "one_exp", "one_exp_2sign", "zero"])
def test_sweep_distributions(lc, oracle, nbits, dist):
    from paper_2009_13003_b200 import synth

    n = (1 << 20) + 4096 * 3 + 5
    base = synth.normal(n, 0.02, DEV, 7)
    if dist in ("one_exp", "one_exp_2sign"):
        base = torch.zeros_like(base)  # so that fl32(cur - base) really lands in one exponent
    cur = base + synth.sweep_delta(dist, n, DEV, 11 + nbits)
    got, _ = assert_stream_parity(lc, oracle, base, cur, nbits)
    assert_recover_parity(lc, oracle, base, [got], inplace=(nbits % 2 == 0))


@pytest.mark.parametrize("logn", [24, 28])
@pytest.mark.parametrize("dist", ["lognormal", "one_exp", "zero"])
def test_sweep_at_benchmarked_sizes(lc, oracle, logn, dist):
    # the sizes of the sweep table (2^24 fits the L2, 2^28 does not), against the oracle on all host cores
    from paper_2009_13003_b200 import synth

    n, nbits = 1 << logn, 5
    base = synth.normal(n, 0.02, DEV, synth.SEED0 + 5)
    if dist == "one_exp":
        base = torch.zeros_like(base)
    cur = base + synth.sweep_delta(dist, n, DEV, synth.SEED0 + 5 + logn)
    bh, ch = to_np(base), to_np(cur)
    got, _ = gpu_compress(lc, base, cur, nbits)
    want = oracle.compress(bh, ch, nbits, threads=ORACLE_THREADS)
    assert got.size == want.size and got.tobytes() == want.tobytes()
    s = torch.from_numpy(got).to(DEV)
    for k in (1, 3):
        out = to_np(lc.recover(base, [s] * k))
        ref = oracle.recover(bh, [want] * k, threads=ORACLE_THREADS)
        assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))


def test_large_deltas_bypass_the_key_plane(lc, oracle):
    # |delta| >= 2 has an exponent field >= 128, which the one-byte key plane cannot hold: the encode
    # pass then takes its keys from base and cur.
    from paper_2009_13003_b200 import synth

    n = 300_000 + 77
    base = synth.normal(n, 1.0, DEV, 31)
    cur = base + synth.normal(n, 40.0, DEV, 32)
    got, _ = assert_stream_parity(lc, oracle, base, cur, 5)
    assert_recover_parity(lc, oracle, base, [got])


def test_high_entropy_symbols(lc, oracle):
    # magnitudes log-uniform over 120 binades, both signs, nbits 8: 255 nearly equiprobable symbols, about
    # 8 bits per element, so chunks outgrow the default shared-memory areas of both passes.
    n = 2_000_003
    g = torch.Generator(device=DEV).manual_seed(33)
    mag = torch.exp2(torch.rand(n, generator=g, device=DEV) * 120.0 - 124.0)
    sgn = torch.randint(0, 2, (n,), generator=g, device=DEV) * 2 - 1
    base = torch.zeros(n, dtype=torch.float32, device=DEV)
    cur = (mag * sgn).to(torch.float32)
    got, _ = assert_stream_parity(lc, oracle, base, cur, 8)
    assert int(np.frombuffer(got[40:48].tobytes(), "<u8")[0]) > 7 * n  # more than 7 bits per element
    assert_recover_parity(lc, oracle, base, [got, got])


def test_deterministic_across_runs(lc):
    base, cur = make_case(5_000_011, 5)
    a, _ = gpu_compress(lc, base, cur, 5)
    for _ in range(3):
        b, _ = gpu_compress(lc, base, cur, 5)
        assert a.tobytes() == b.tobytes()


def _fibonacci_case(nsyms, sort_rare_first, seed=3):
    """Deltas whose bucket counts follow the Fibonacci numbers: the deepest possible Huffman tree."""
    fib = [1, 1]
    while len(fib) < nsyms:
        fib.append(fib[-1] + fib[-2])
    g = torch.Generator(device="cpu").manual_seed(seed)
    parts = []
    for j, cnt in enumerate(fib):  # j = 0 rarest; give rarer symbols larger exponents so they are all kept
        E = 140 - j
        mant = torch.randint(0, 1 << 23, (cnt,), generator=g, dtype=torch.int32)
        parts.append(mant | (E << 23))
    bits = torch.cat(parts)
    if not sort_rare_first:
        bits = bits[torch.randperm(bits.numel(), generator=g)]
    cur = bits.view(torch.float32).to(DEV)
    return torch.zeros_like(cur), cur


@pytest.mark.parametrize("rare_first", [False, True])
def test_long_codes_and_oversized_chunks(lc, oracle, rare_first):
    # 35 Fibonacci-weighted buckets -> code lengths up to 34 bits (> 32: the split-code path of the
    # encoder, > lookup width: the canonical search of the decoder). With the rare symbols first the
    # leading chunks average more bits per element than the encoder's staging area holds.
    base, cur = _fibonacci_case(35, rare_first)
    got, want = assert_stream_parity(lc, oracle, base, cur, 6)
    assert got[20] == 34
    assert_recover_parity(lc, oracle, base, [got])


def test_medium_long_codes(lc, oracle):
    base, cur = _fibonacci_case(24, False)  # lengths up to 23: longer than the lookup, shorter than 32
    got, _ = assert_stream_parity(lc, oracle, base, cur, 5)
    assert got[20] == 23
    assert_recover_parity(lc, oracle, base, [got])


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 8])
def test_chain_recover(lc, oracle, k):
    # Algorithm 1: each compress uses the tracked state as base; recovering all streams from u_0
    # reproduces the tracked state bit for bit.
    from paper_2009_13003_b200 import synth

    n = 300_007
    u0 = synth.normal(n, 0.05, DEV, 21)
    u, tracked, streams = u0.clone(), u0.clone(), []
    for t in range(k):
        u = u + synth.normal(n, 1e-3, DEV, 22 + t)
        s, _ = assert_stream_parity(lc, oracle, tracked, u, 3)
        streams.append(s)
        tracked = lc.recover(tracked, [torch.from_numpy(s).to(DEV)])
    out = assert_recover_parity(lc, oracle, u0, streams)
    assert np.array_equal(out.view(np.uint32), to_np(tracked).view(np.uint32))


def test_config_lenet5(lc, oracle):
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS["lenet5"]
    base = synth.base_state(cfg, DEV)
    cur = base + synth.snapshot_delta(cfg, 1, DEV)
    got, _ = assert_stream_parity(lc, oracle, base, cur, cfg.nbits)
    assert_recover_parity(lc, oracle, base, [got])


def test_config_resnet18_chain(lc, oracle):
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS["resnet18"]
    u0 = synth.base_state(cfg, DEV)
    u, tracked, streams = u0.clone(), u0.clone(), []
    for t in range(1, cfg.chain + 1):
        u = u + synth.snapshot_delta(cfg, t, DEV)
        s, _ = assert_stream_parity(lc, oracle, tracked, u, cfg.nbits)
        streams.append(s)
        tracked = lc.recover(tracked, [torch.from_numpy(s).to(DEV)])
    # ten streams: two chained calls of at most LC_MAX_CHAIN
    dev_streams = [torch.from_numpy(s).to(DEV) for s in streams]
    mid = lc.recover(u0, dev_streams[:8])
    out = lc.recover(mid, dev_streams[8:])
    assert np.array_equal(to_np(out).view(np.uint32), to_np(tracked).view(np.uint32))
    want = oracle.recover(oracle.recover(to_np(u0), streams[:8]), streams[8:])
    assert np.array_equal(to_np(out).view(np.uint32), want.view(np.uint32))


def test_config_vgg16(lc, oracle):
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS["vgg16"]
    base = synth.base_state(cfg, DEV)
    cur = base + synth.snapshot_delta(cfg, 1, DEV)
    got, _ = assert_stream_parity(lc, oracle, base, cur, cfg.nbits)
    assert_recover_parity(lc, oracle, base, [got])


def test_config_xfmr1p3b_full_size(lc, oracle):
    """The benchmark's workload at full size: 1,315,575,808 elements, nbits 5, chain of 4.

    Every stream of the chain is compared byte for byte with the oracle's (coded with all host cores), after
    the statistics and the table, so that a failure names the step; sampled chunks are also coded one by one;
    the recovered state is compared in full against Algorithm 1 step 7 computed directly on the CPU.
    """
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS["xfmr1p3b"]
    n, nbits = cfg.n, cfg.nbits
    u0 = synth.base_state(cfg, DEV)
    u0_h = to_np(u0)
    tracked, tracked_h = u0.clone(), u0_h.copy()
    u = u0.clone()
    rng = np.random.default_rng(0)
    nchunks = (n + 4095) // 4096
    stream_buf = [lc.alloc_stream(n, nbits, DEV) for _ in range(cfg.chain)]
    ws = lc.alloc_workspace(n, DEV)
    streams = []
    for t in range(1, cfg.chain + 1):
        u += synth.snapshot_delta(cfg, t, DEV)
        lc.compress_async(tracked, u, nbits, stream_buf[t - 1], ws)
        assert lc.last_status(ws) == 0
        info = lc.stream_info(stream_buf[t - 1])
        s = stream_buf[t - 1][: info.total_bytes]
        streams.append(s)
        u_h = to_np(u)
        # statistics and table, in full
        count, mmin, mmax = lc.debug_bins(ws)
        ocount, omin, omax = oracle.bins(tracked_h, u_h)
        assert np.array_equal(count, ocount) and np.array_equal(mmin, omin) and np.array_equal(mmax, omax)
        tab = oracle.table(tracked_h, u_h, nbits)
        nsym = len(tab["key"])
        head = to_np(s[: 64 + 16 * nsym])
        assert int(np.frombuffer(head[16:20].tobytes(), "<u4")[0]) == nsym
        ent = np.frombuffer(head[64:].tobytes(), dtype=[("key", "<u2"), ("len", "u1"), ("pad", "u1"),
                                                         ("rep", "<u4"), ("count", "<u8")])
        assert np.array_equal(ent["key"], tab["key"].astype(np.uint16))
        assert np.array_equal(ent["len"], tab["len"].astype(np.uint8))
        assert np.array_equal(ent["rep"], tab["rep"].view(np.uint32))
        assert np.array_equal(ent["count"], tab["count"])
        payload_bits = int((tab["count"] * tab["len"].astype(np.uint64)).sum())
        assert info.payload_bits == payload_bits and info.max_len == int(tab["len"].max())
        # indices: properties that hold for the whole stream
        ci_off = 64 + 16 * nsym
        li_off = ci_off + 8 * (nchunks + 1)
        chunk_off = to_np(s[ci_off:li_off]).view("<u8")
        lane_bits = to_np(s[li_off: li_off + 64 * nchunks]).view("<u2").reshape(nchunks, 32)
        assert int(lane_bits.sum(dtype=np.uint64)) == payload_bits
        sizes = ((lane_bits.sum(1, dtype=np.int64) + 7) // 8 + 15) // 16 * 16
        assert chunk_off[0] == 0 and np.array_equal(np.diff(chunk_off.astype(np.int64)), sizes)
        assert info.payload_offset + int(chunk_off[-1]) == info.total_bytes
        # payload: sampled chunks, coded by the oracle
        ids = np.unique(np.concatenate([[0, 1, nchunks - 2, nchunks - 1], rng.integers(0, nchunks, 48)]))
        olane, opay = oracle.compress_chunks(tracked_h, u_h, nbits, ids)
        for k, c in enumerate(ids.tolist()):
            assert np.array_equal(lane_bits[c], olane[k]), c
            lo = info.payload_offset + int(chunk_off[c])
            assert to_np(s[lo: lo + opay[k].size]).tobytes() == opay[k].tobytes(), c
        # the whole stream
        want = oracle.compress(tracked_h, u_h, nbits, threads=ORACLE_THREADS)
        assert want.size == info.total_bytes
        got = to_np(s)
        step = 1 << 28
        for lo in range(0, want.size, step):
            assert got[lo: lo + step].tobytes() == want[lo: lo + step].tobytes(), "stream %d differs near byte %d" % (t, lo)
        del want, got
        # tracked state: GPU recover vs step 7 computed directly
        tracked_h = oracle.apply_quantized(tracked_h, u_h, nbits)
        lc.recover(tracked, [s], out=tracked, workspace=ws)
        del u_h
    got = to_np(lc.recover(u0, streams, workspace=ws))
    assert np.array_equal(got.view(np.uint32), tracked_h.view(np.uint32))
    assert np.array_equal(to_np(tracked).view(np.uint32), tracked_h.view(np.uint32))


# ---------------------------------------------------------------- error paths (no fault, only status)


def test_argument_errors(lc):
    base, cur = make_case(5000, 1)
    ws = lc.alloc_workspace(5000, DEV)
    st = lc.alloc_stream(5000, 4, DEV)
    L = lc.lib()
    cs = None
    assert L.lc_compress(base.data_ptr(), cur.data_ptr(), 5000, 0, st.data_ptr(), st.numel(), ws.data_ptr(), ws.numel(), cs) == lc.ERR_ARG
    assert L.lc_compress(base.data_ptr(), cur.data_ptr(), 5000, 10, st.data_ptr(), st.numel(), ws.data_ptr(), ws.numel(), cs) == lc.ERR_ARG
    assert L.lc_compress(None, cur.data_ptr(), 5000, 4, st.data_ptr(), st.numel(), ws.data_ptr(), ws.numel(), cs) == lc.ERR_ARG
    assert L.lc_compress(base.data_ptr() + 4, cur.data_ptr(), 4999, 4, st.data_ptr(), st.numel(), ws.data_ptr(), ws.numel(), cs) == lc.ERR_ARG
    assert L.lc_compress(base.data_ptr(), cur.data_ptr(), 5000, 4, st.data_ptr(), st.numel() - 1, ws.data_ptr(), ws.numel(), cs) == lc.ERR_CAPACITY
    assert L.lc_compress(base.data_ptr(), cur.data_ptr(), 5000, 4, st.data_ptr(), st.numel(), ws.data_ptr(), ws.numel() - 1, cs) == lc.ERR_CAPACITY
    assert L.lc_compress(base.data_ptr(), cur.data_ptr(), 1 << 32, 4, st.data_ptr(), st.numel(), ws.data_ptr(), ws.numel(), cs) == lc.ERR_ARG
    torch.cuda.synchronize()


def test_nonfinite_delta_is_reported(lc, oracle):
    base, cur = make_case(100_000, 2)
    for bad in (float("inf"), float("-inf"), float("nan")):
        c2 = cur.clone()
        c2[77_777] = bad
        with pytest.raises(lc.LCError) as e:
            gpu_compress(lc, base, c2, 4)
        assert e.value.code == lc.ERR_NONFINITE
        with pytest.raises(oracle.OracleError) as eo:
            oracle.compress(to_np(base), to_np(c2), 4)
        assert eo.value.code == oracle.ERR_NONFINITE
    # the workspace is usable again afterwards
    assert_stream_parity(lc, oracle, base, cur, 4)


def test_corrupted_streams_are_rejected_not_faulting(lc, oracle):
    n = 200_000
    base, cur = make_case(n, 3)
    good, _ = gpu_compress(lc, base, cur, 4)

    def status_of(stream_np, nn=n, b=base):
        s = torch.from_numpy(stream_np.copy()).to(DEV)
        ws = lc.alloc_workspace(0, DEV)
        out = torch.empty(nn, dtype=torch.float32, device=DEV)
        lc.recover_async(b[:nn].contiguous(), [s], out, ws)
        return lc.last_status(ws)

    def mutated(off, val):
        m = good.copy()
        m[off] = val
        return m

    assert status_of(good) == 0
    assert status_of(mutated(0, ord("X"))) == lc.ERR_FORMAT       # magic
    assert status_of(mutated(4, 2)) == lc.ERR_FORMAT              # version
    assert status_of(mutated(6, 10)) == lc.ERR_FORMAT             # nbits
    assert status_of(mutated(16, 200)) == lc.ERR_FORMAT           # nsym
    assert status_of(mutated(24, 1)) == lc.ERR_FORMAT             # chunk_elems
    assert status_of(mutated(64 + 16 + 2, 1)) == lc.ERR_FORMAT    # a code length: Kraft / bit count
    assert status_of(mutated(48, (int(good[48]) + 16) % 256)) == lc.ERR_FORMAT  # total_bytes
    assert status_of(good[:-16]) == lc.ERR_FORMAT                 # truncated buffer
    assert status_of(good, nn=n - 1) == lc.ERR_MISMATCH
    # damaged chunk index entry (offset beyond the payload): flagged, no fault
    nsym = int(np.frombuffer(good[16:20].tobytes(), "<u4")[0])
    m = good.copy()
    m[64 + 16 * nsym + 8 + 5] = 0x7F
    assert status_of(m) == lc.ERR_FORMAT
    # damaged payload and lane index: output unspecified, but the call completes and the next is fine
    po = int(np.frombuffer(good[56:64].tobytes(), "<u8")[0])
    m = good.copy()
    m[po: po + 4096] = 0xFF
    m[po - 640: po - 600] = 0xFF
    assert status_of(m) in (0, lc.ERR_FORMAT)
    torch.cuda.synchronize()
    assert status_of(good) == 0


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("n,k", [(1_234_567, 2), (1_234_567, 6), (130 * 4096, 1), (50_001, 3), (0, 1)])
def test_host_buffer_entry_points(lc, oracle, n, k, pinned):
    """Large vectors go through lc_recover_host in slices of whole chunks (copies in both directions overlapped with
    the decode of the slice between them), small ones in one piece; a chain above four streams takes two passes per
    slice. All of it must give the oracle's values."""
    nbits = 4
    base, cur = make_case(n, 9)
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)  # pageable buffers make the copies synchronous
    bh, ch = pin(base.cpu()), pin(cur.cpu())
    arena = torch.empty(lc.host_arena_bytes(n, nbits, k), dtype=torch.uint8, device=DEV)
    sh = pin(torch.empty(lc.stream_bound(n, nbits), dtype=torch.uint8))
    size = lc.compress_host(bh, ch, nbits, sh, arena)
    want = oracle.compress(bh.numpy(), ch.numpy(), nbits)
    assert sh[:size].numpy().tobytes() == want.tobytes()
    oh = pin(torch.full((n,), 7.0, dtype=torch.float32))
    lc.recover_host(bh, [sh[:size]] * k, oh, arena)
    assert np.array_equal(oh.numpy().view(np.uint32), oracle.recover(bh.numpy(), [want] * k).view(np.uint32))
    if n:
        bad = sh[:size].clone()
        bad[0] = 0
        with pytest.raises(Exception):
            lc.recover_host(bh, [sh[:size]] * (k - 1) + [bad], oh, arena)
        lc.recover_host(bh, [sh[:size]] * k, oh, arena)


def test_more_than_2_31_elements(lc, oracle):
    """A vector of 2^31 + 3 * 4096 + 5 elements (8.6 GB of fp32, ragged tail): every element index, chunk number and
    byte offset beyond 32 bits' signed range. The stream is compared byte for byte with the oracle's (all host
    cores), the recovered state bit for bit."""
    from paper_2009_13003_b200 import synth

    n, nbits = (1 << 31) + 3 * 4096 + 5, 4
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GB of free device memory")
    base = synth.normal(n, 0.02, DEV, 31)
    cur = base + synth.laplace(n, 1e-3, DEV, 32)
    ws, sbuf = lc.alloc_workspace(n, DEV), lc.alloc_stream(n, nbits, DEV)
    lc.compress_async(base, cur, nbits, sbuf, ws)
    assert lc.last_status(ws) == 0
    info = lc.stream_info(sbuf)
    assert info.valid == 1 and info.n == n and info.nchunks == (n + 4095) // 4096
    base_h, cur_h = to_np(base), to_np(cur)
    want = oracle.compress(base_h, cur_h, nbits, threads=ORACLE_THREADS)
    assert want.size == info.total_bytes
    got = to_np(sbuf[: info.total_bytes])
    step = 1 << 28
    for lo in range(0, want.size, step):
        assert got[lo: lo + step].tobytes() == want[lo: lo + step].tobytes(), "stream differs near byte %d" % lo
    del got, cur_h
    out = lc.recover(base, [sbuf[: info.total_bytes]], out=cur, workspace=ws)  # cur is no longer needed
    want_out = oracle.recover(base_h, [want], threads=ORACLE_THREADS)
    assert np.array_equal(to_np(out).view(np.uint32), want_out.view(np.uint32))
