"""Pins of the CPU oracle to facts fixed by the paper and by mathematics (CPU only).

Each test is chosen so that a plausible mistake in one step of the oracle (a dropped term, a wrong
sign, index, order or rounding) fails it. Nothing here calls the CUDA path.
"""
import itertools
import math

import numpy as np
import pytest

from conftest import load_golden


def f32(bits):
    return np.array(bits, np.uint32).view(np.float32)


# ---------------------------------------------------------------- hand-worked golden streams


@pytest.mark.parametrize("name", ["ten_elements_nbits2.txt", "skew16_nbits3.txt"])
def test_golden_stream_bytes(oracle, name):
    g = load_golden(name)
    base = np.zeros(g["cur"].size, np.float32)
    s = oracle.compress(base, g["cur"], g["nbits"])
    assert s.tobytes() == g["stream"].tobytes()
    out = oracle.recover(base, [g["stream"]])
    assert out.view(np.uint32).tolist() == g["recovered"].view(np.uint32).tolist()


def test_paper_size_model_example(oracle):
    # Section 3.1.1 worked example: n = 10, b = 32, k = 5 -> 190 bits, rate 1.68.
    bits = oracle.model_bits(10, 5, 32)
    assert bits == 190
    assert round(10 * 32 / bits, 2) == 1.68
    # and the 2-bit promotion of that example leaves 4 buckets of 2 bits each.
    assert oracle.model_bits(10, 4, 32) == 10 * 2 + 4 * 32


def test_paper_example_shape(oracle):
    # Figure 1 text: 10 elements, 5 buckets; 2-bit promotion keeps 3 and merges 2 into the zero bucket.
    g = load_golden("ten_elements_nbits2.txt")
    base = np.zeros(10, np.float32)
    count, _, _ = oracle.bins(base, g["cur"])
    assert int((count > 0).sum()) == 5
    t = oracle.table(base, g["cur"], 2)
    assert len(t["key"]) == 4 and t["rep"][0] == 0.0 and int(t["count"][0]) == 2


# ---------------------------------------------------------------- O1-O3: delta and buckets


def test_bins_hand_vector(oracle):
    # known bit patterns: 1.0, 1.5, -0.75, smallest normal, a subnormal, +0, -0, and a delta that is
    # only representable after the fp32 subtract rounds.
    cur = f32([0x3F800000, 0x3FC00000, 0xBF400000, 0x00800000, 0x00000001, 0x00000000, 0x80000000])
    base = np.zeros(cur.size, np.float32)
    count, mmin, mmax = oracle.bins(base, cur)
    exp = {127: 2, 256 + 126: 1, 1: 1, 0: 2, 256: 1}
    for key in range(512):
        assert int(count[key]) == exp.get(key, 0), key
    assert (mmin[127], mmax[127]) == (0, 0x400000)
    assert (mmin[256 + 126], mmax[256 + 126]) == (0x400000, 0x400000)
    assert (mmin[0], mmax[0]) == (0, 1)  # +0 and the subnormal share E = 0, s = 0


def test_delta_is_fp32_subtract(oracle):
    # cur - base must be rounded once to fp32: 1 + 2^-24 is not representable, and (1+2^-23) - 2^-24
    # rounds to even.
    base = np.array([np.float32(2.0 ** -24)], np.float32)
    cur = f32([0x3F800001])
    d = (cur - base).view(np.uint32)[0]
    count, mmin, mmax = oracle.bins(base, cur)
    key = int(d >> 23)
    assert count[key] == 1 and mmin[key] == (d & 0x7FFFFF) == mmax[key]


def test_bins_against_sort_and_group(oracle):
    rng = np.random.default_rng(5)
    n = 20011
    base = rng.normal(0, 0.02, n).astype(np.float32)
    cur = (base + rng.laplace(0, 1e-3, n).astype(np.float32)).astype(np.float32)
    cur[::97] = base[::97]  # exact zeros
    count, mmin, mmax = oracle.bins(base, cur)
    bits = (cur - base).view(np.uint32)
    order = np.sort(bits)
    keys = order >> 23
    assert int(count.sum()) == n
    for key in np.unique(keys):
        grp = order[keys == key]
        assert int(count[key]) == grp.size
        assert int(mmin[key]) == int(grp[0] & 0x7FFFFF)
        assert int(mmax[key]) == int(grp[-1] & 0x7FFFFF)
    assert all(count[k] == 0 for k in range(512) if k not in set(keys.tolist()))


# ---------------------------------------------------------------- O4: priority promotion


def _vector_with_keys(keys):
    """One element per (s, E) key, mantissa 0."""
    bits = [((k >> 8) << 31) | ((k & 255) << 23) for k in keys]
    return f32(bits)


def test_selection_order_and_limit(oracle):
    keys = [100, 256 + 100, 130, 256 + 131, 90, 256 + 90, 1, 254, 0, 256]  # includes E=0 keys
    cur = _vector_with_keys(keys)
    base = np.zeros(cur.size, np.float32)
    full = [254, 256 + 131, 130, 100, 256 + 100, 90, 256 + 90, 1]  # E desc, + before -
    for nbits in range(1, 9):
        t = oracle.table(base, cur, nbits)
        K = min(2 ** nbits - 1, len(full))
        assert t["key"].tolist() == [0] + full[:K]
        assert len(t["key"]) <= 2 ** nbits
        assert int(t["count"][0]) == len(keys) - K
        sym = oracle.symbols(base, cur, nbits)
        for i, k in enumerate(keys):
            assert sym[i] == (full.index(k) + 1 if k in full[:K] else 0)


def test_subnormals_and_zero_never_selected(oracle):
    cur = f32([0x00000001, 0x807FFFFF, 0x00000000, 0x80000000])
    t = oracle.table(np.zeros(4, np.float32), cur, 8)
    assert t["key"].tolist() == [0] and int(t["count"][0]) == 4 and t["len"].tolist() == [0]


def test_nonfinite_rejected(oracle):
    for bad in (0x7F800000, 0xFF800000, 0x7FC00000):
        cur = f32([0x3F800000, bad])
        with pytest.raises(oracle.OracleError) as e:
            oracle.compress(np.zeros(2, np.float32), cur, 4)
        assert e.value.code == oracle.ERR_NONFINITE


# ---------------------------------------------------------------- O5: representative


def _int_midrange(s, E, m0, m1):
    t = m0 + m1
    mr = t >> 1
    if (t & 1) and (mr & 1):
        mr += 1
    return (s << 31) | (E << 23) | mr


def test_midrange_equals_integer_formula(oracle):
    rng = np.random.default_rng(11)
    cases = [(0, 254, 0x7FFFFE, 0x7FFFFF), (1, 254, 0x7FFFFF, 0x7FFFFF), (0, 1, 0, 1), (1, 1, 1, 2),
             (0, 127, 1, 2), (0, 127, 1, 4), (0, 127, 3, 4), (0, 127, 0x7FFFFD, 0x7FFFFE)]
    for _ in range(4000):
        m0, m1 = sorted(rng.integers(0, 1 << 23, 2).tolist())
        cases.append((int(rng.integers(0, 2)), int(rng.integers(1, 255)), m0, m1))
    for s, E, m0, m1 in cases:
        lo = f32([(s << 31) | (E << 23) | m0])[0]
        hi = f32([(s << 31) | (E << 23) | m1])[0]
        vmin, vmax = (hi, lo) if s else (lo, hi)
        rep = oracle.midrange(vmin, vmax)
        assert int(np.float32(rep).view(np.uint32)) == _int_midrange(s, E, m0, m1), (s, E, m0, m1)
        assert vmin <= rep <= vmax


def test_rep_single_element_bucket_is_the_element(oracle):
    cur = f32([0x3DCCCCCD, 0xBDCCCCCD, 0x3A83126F])
    t = oracle.table(np.zeros(3, np.float32), cur, 4)
    assert sorted(t["rep"][1:].view(np.uint32).tolist()) == sorted(cur.view(np.uint32).tolist())


# ---------------------------------------------------------------- O6: Huffman


def _brute_force_cost(counts, max_len):
    best = None
    for lens in itertools.product(range(1, max_len + 1), repeat=len(counts)):
        if sum(2.0 ** -l for l in lens) <= 1.0 + 1e-12:
            cost = sum(c * l for c, l in zip(counts, lens))
            best = cost if best is None else min(best, cost)
    return best


def test_huffman_optimal_vs_brute_force(oracle):
    rng = np.random.default_rng(3)
    trials = []
    for k in range(2, 7):
        for _ in range(12):
            trials.append(rng.integers(1, 40, k).tolist())        # random
            trials.append(rng.integers(1, 4, k).tolist())         # tie-heavy
        trials.append([1] * k)
        trials.append([2 ** i for i in range(k)])
    for counts in trials:
        ln, code = oracle.huffman(counts)
        cost = sum(c * int(l) for c, l in zip(counts, ln))
        assert cost == _brute_force_cost(counts, len(counts)), counts


def _kraft_and_prefix_free(ln, code):
    used = [(int(l), int(c)) for l, c in zip(ln, code) if l > 0]
    assert sum(2 ** (64 - l) for l, _ in used) == 2 ** 64  # Kraft equality, exact
    strs = [format(c, "0%db" % l) for l, c in used]
    for a, b in itertools.permutations(strs, 2):
        assert not b.startswith(a)


def test_huffman_kraft_entropy_prefix(oracle):
    rng = np.random.default_rng(4)
    for k in (2, 3, 5, 8, 16, 31, 32, 64, 200, 256):
        for scale in (1.0, 1e3, 1e9):
            counts = np.maximum(1, (rng.pareto(1.2, k) * scale).astype(np.uint64))
            ln, code = oracle.huffman(counts)
            _kraft_and_prefix_free(ln, code)
            p = counts / counts.sum()
            H = float(-(p * np.log2(p)).sum())
            Lbar = float((p * ln).sum())
            assert H - 1e-9 <= Lbar < H + 1


def test_huffman_textbook_cases(oracle):
    for j in range(1, 9):  # 2^j equal counts -> all lengths j
        ln, _ = oracle.huffman([7] * (2 ** j))
        assert ln.tolist() == [j] * (2 ** j)
    ln, _ = oracle.huffman([1, 1, 2, 4, 8, 16])  # dyadic
    assert ln.tolist() == [5, 5, 4, 3, 2, 1]
    fib = [1, 1, 2, 3, 5, 8, 13, 21, 34, 55, 89, 144]  # maximal depth
    ln, _ = oracle.huffman(fib)
    assert ln.tolist() == [11, 11, 10, 9, 8, 7, 6, 5, 4, 3, 2, 1]
    big = [1, 1]
    while len(big) < 45:
        big.append(big[-1] + big[-2])
    ln, code = oracle.huffman(big)  # total < 2^32, depth 44: codes longer than 32 bits
    assert int(ln.max()) == 44 and sum(big) < 2 ** 32
    _kraft_and_prefix_free(ln, code)


def test_huffman_tie_break_and_canonical_hand_case(oracle):
    # five equal counts, worked by hand with the two-queue rule (leaf before internal node on ties):
    # (a+b)=2, (c+d)=2, e+(ab)=3, (cd)+3=5 -> a,b depth 3; c,d,e depth 2.
    ln, code = oracle.huffman([1, 1, 1, 1, 1])
    assert ln.tolist() == [3, 3, 2, 2, 2]
    assert code.tolist() == [0b110, 0b111, 0b00, 0b01, 0b10]
    # zero-count symbols take no part and get length 0
    ln, code = oracle.huffman([0, 5, 0, 5, 0])
    assert ln.tolist() == [0, 1, 0, 1, 0] and code.tolist() == [0, 0, 0, 1, 0]
    # one used symbol -> length 0
    ln, _ = oracle.huffman([0, 9, 0])
    assert ln.tolist() == [0, 0, 0]


def test_canonical_codes_increase(oracle):
    rng = np.random.default_rng(8)
    counts = rng.integers(1, 10 ** 6, 100)
    ln, code = oracle.huffman(counts)
    order = sorted(range(100), key=lambda j: (ln[j], j))
    vals = [int(code[j]) << (int(ln.max()) - int(ln[j])) for j in order]  # left-aligned
    assert all(a < b for a, b in zip(vals, vals[1:]))


# ---------------------------------------------------------------- O7: stream


def _random_case(rng, n, scale=1e-3):
    base = rng.normal(0, 0.02, n).astype(np.float32)
    cur = (base + rng.laplace(0, scale, n).astype(np.float32)).astype(np.float32)
    return base, cur


@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 127, 128, 129, 4095, 4096, 4097, 3 * 4096 + 77, 70001])
@pytest.mark.parametrize("nbits", [1, 3, 8])
def test_roundtrip_symbols_and_sizes(oracle, n, nbits):
    rng = np.random.default_rng(n * 10 + nbits)
    base, cur = _random_case(rng, n)
    s = oracle.compress(base, cur, nbits)
    assert s.size <= oracle.stream_bound(n, nbits)
    t = oracle.table(base, cur, nbits)
    sym = oracle.symbols(base, cur, nbits)
    assert np.array_equal(oracle.decode_symbols(s, n), sym)
    # header fields
    payload_bits = int(np.frombuffer(s[40:48].tobytes(), "<u8")[0])
    assert payload_bits == int((t["count"] * t["len"].astype(np.uint64)).sum())
    assert int(np.frombuffer(s[48:56].tobytes(), "<u8")[0]) == s.size
    nchunks = (n + 4095) // 4096
    nsym = len(t["key"])
    ci = 64 + 16 * nsym
    li = ci + 8 * (nchunks + 1)
    chunk_off = np.frombuffer(s[ci:li].tobytes(), "<u8")
    lane_bits = np.frombuffer(s[li:li + 64 * nchunks].tobytes(), "<u2").reshape(nchunks, 32)
    assert int(lane_bits.sum()) == payload_bits
    sizes = np.diff(chunk_off)
    assert np.array_equal(sizes, ((lane_bits.sum(1).astype(np.int64) + 7) // 8 + 15) // 16 * 16)
    # lane lengths recomputed from the symbols and the element order of the format
    ln = t["len"]
    for c in range(nchunks):
        for lane in (0, 1, 31):
            idx = [4096 * c + 128 * j + 4 * lane + e for j in range(32) for e in range(4)]
            idx = [i for i in idx if i < n]
            assert int(lane_bits[c, lane]) == int(sum(int(ln[sym[i]]) for i in idx))


def test_payload_bits_by_independent_bit_writer(oracle):
    # re-create one chunk's payload from (symbols, codes) with python string concatenation.
    rng = np.random.default_rng(21)
    n = 4096 + 600
    base, cur = _random_case(rng, n)
    s = oracle.compress(base, cur, 4)
    t = oracle.table(base, cur, 4)
    sym = oracle.symbols(base, cur, 4)
    nsym, nchunks = len(t["key"]), 2
    ci = 64 + 16 * nsym
    li = ci + 8 * (nchunks + 1)
    po = (li + 64 * nchunks + 15) // 16 * 16
    chunk_off = np.frombuffer(s[ci:li].tobytes(), "<u8")
    for c in range(nchunks):
        bits = ""
        for lane in range(32):
            for j in range(32):
                for e in range(4):
                    i = 4096 * c + 128 * j + 4 * lane + e
                    if i < n and t["len"][sym[i]] > 0:
                        bits += format(int(t["code"][sym[i]]), "0%db" % int(t["len"][sym[i]]))
        nbytes = ((len(bits) + 7) // 8 + 15) // 16 * 16
        bits = bits.ljust(nbytes * 8, "0")
        words = [int(bits[w:w + 32], 2) for w in range(0, len(bits), 32)]
        expect = np.array(words, "<u4").tobytes()
        got = s[po + int(chunk_off[c]): po + int(chunk_off[c + 1])].tobytes()
        assert got == expect


def test_single_symbol_and_empty(oracle):
    base = np.linspace(-1, 1, 5000).astype(np.float32)
    s = oracle.compress(base, base, 5)  # all-zero delta
    assert int(np.frombuffer(s[40:48].tobytes(), "<u8")[0]) == 0  # no payload bits
    assert s[20] == 0  # max_len
    out = oracle.recover(base, [s])
    assert np.array_equal(out.view(np.uint32), (base + np.float32(0)).view(np.uint32))
    # one exponent, one sign, no zeros: the single used symbol is symbol 1
    cur = (1.0 + np.random.default_rng(0).random(3000)).astype(np.float32)
    s = oracle.compress(np.zeros(3000, np.float32), cur, 2)
    assert np.all(oracle.decode_symbols(s, 3000) == 1)
    s0 = oracle.compress(np.zeros(0, np.float32), np.zeros(0, np.float32), 3)
    assert s0.size == 64 + 16 + 8 + 8  # header, one table entry, chunk_off[0], padding to 16
    assert oracle.recover(np.zeros(0, np.float32), [s0]).size == 0


# ---------------------------------------------------------------- O8: recovery


def test_recover_equals_base_plus_rep(oracle):
    rng = np.random.default_rng(31)
    n = 30000
    base, cur = _random_case(rng, n)
    base[:5] = f32([0x80000000] * 5)  # -0.0 base: adding the +0 representative gives +0.0
    cur[:5] = base[:5]
    for nbits in (2, 4, 6):
        s = oracle.compress(base, cur, nbits)
        t = oracle.table(base, cur, nbits)
        sym = oracle.symbols(base, cur, nbits)
        expect = base + t["rep"][sym]
        out = oracle.recover(base, [s])
        assert np.array_equal(out.view(np.uint32), expect.view(np.uint32))
        assert out[:5].view(np.uint32).tolist() == [0] * 5
        # error bound of exponent quantization: kept elements stay within half a binade's width
        d = cur - base
        dq = t["rep"][sym]
        kept = sym > 0
        e = np.floor(np.log2(np.abs(d[kept])))
        assert np.all(np.abs(dq[kept].astype(np.float64) - d[kept]) < 2.0 ** (e - 1) + 1e-300)
        assert np.all(dq[~kept] == 0)
        assert np.all(np.sign(dq[kept]) == np.sign(d[kept]))


def test_chain_identity(oracle):
    # Algorithm 1: tracked state u~_t = u~_{t-1} + quantized delta; recovery from u_0 and all streams
    # reproduces u~_t bit for bit.
    rng = np.random.default_rng(41)
    n = 9001
    u0 = rng.normal(0, 0.05, n).astype(np.float32)
    u, tracked, streams = u0.copy(), u0.copy(), []
    for t in range(5):
        u = (u + rng.normal(0, 1e-3, n).astype(np.float32)).astype(np.float32)
        s = oracle.compress(tracked, u, 3)
        streams.append(s)
        tracked = oracle.recover(tracked, [s])
        out = oracle.recover(u0, streams)
        assert np.array_equal(out.view(np.uint32), tracked.view(np.uint32))
    # error feedback keeps the tracked state near the true state
    assert float(np.abs(tracked - u).max()) < 5e-3


def test_compress_of_identical_states(oracle):
    x = np.random.default_rng(2).normal(0, 1, 10000).astype(np.float32)
    s = oracle.compress(x, x, 4)
    assert np.all(oracle.decode_symbols(s, x.size) == 0)


# ---------------------------------------------------------------- malformed streams


def test_reader_rejects_corruption(oracle):
    rng = np.random.default_rng(51)
    n = 10000
    base, cur = _random_case(rng, n)
    good = oracle.compress(base, cur, 4)
    assert oracle.recover(base, [good]).size == n

    def expect(mut, code):
        bad = good.copy()
        mut(bad)
        with pytest.raises(oracle.OracleError) as e:
            oracle.recover(base, [bad])
        assert e.value.code == code

    def setb(off, val):
        return lambda b: b.__setitem__(off, val)

    expect(setb(0, ord("X")), oracle.ERR_FORMAT)     # magic
    expect(setb(4, 2), oracle.ERR_FORMAT)            # version
    expect(setb(6, 10), oracle.ERR_FORMAT)           # nbits
    expect(setb(7, 16), oracle.ERR_FORMAT)           # flags
    expect(setb(16, 200), oracle.ERR_FORMAT)         # nsym > 2^nbits
    expect(setb(24, 1), oracle.ERR_FORMAT)           # chunk_elems
    expect(setb(64 + 16 + 2, 1), oracle.ERR_FORMAT)  # a code length changed: Kraft / payload_bits
    expect(setb(48, (int(good[48]) + 16) % 256), oracle.ERR_FORMAT)  # total_bytes
    with pytest.raises(oracle.OracleError) as e:
        oracle.recover(base, [good[:-16]])           # truncated buffer
    assert e.value.code == oracle.ERR_FORMAT
    with pytest.raises(oracle.OracleError) as e:
        oracle.recover(base[:-1], [good])
    assert e.value.code == oracle.ERR_MISMATCH


def test_ratio_ranges_on_synthetic_deltas(oracle):
    # Section 4.3 reports E+P+H below 5 % (2-bit) and 10 % (3-bit) on its training deltas; a
    # concentrated synthetic delta must land in the same region (sanity range, not an acceptance test).
    rng = np.random.default_rng(61)
    n = 200000
    base = rng.normal(0, 0.02, n).astype(np.float32)
    cur = (base + rng.normal(0, 1e-3, n).astype(np.float32)).astype(np.float32)
    for nbits, limit in ((2, 0.05), (3, 0.10)):
        s = oracle.compress(base, cur, nbits)
        payload_bits = int(np.frombuffer(s[40:48].tobytes(), "<u8")[0])
        assert payload_bits / (32 * n) < limit
        assert payload_bits <= n * nbits


# ---------------------------------------------------------------- helpers the GPU parity tests lean on


def _helper_cases():
    rng = np.random.default_rng(61)
    cases = []
    for n, nbits in ((1, 1), (5, 3), (4097, 3), (3 * 4096 + 77, 8), (70001, 1), (20000, 3)):
        base, cur = _random_case(rng, n)
        cases.append((base, cur, nbits))
    # a -0.0 base under an unchanged element, and deltas over a wide range of exponents (fields above 127 too)
    n = 9000
    base = rng.normal(0, 1.0, n).astype(np.float32)
    base[:7] = f32([0x80000000] * 7)
    cur = (base + (rng.normal(0, 1, n) * np.exp2(rng.integers(-40, 20, n))).astype(np.float32)).astype(np.float32)
    cur[:7] = base[:7]
    cases.append((base, cur, 3))
    cases.append((base, cur, 8))
    return cases


def test_apply_quantized_is_recover_of_compress(oracle):
    # Algorithm 1 step 7 computed directly must be what decoding the stream and adding gives, bit for bit.
    for base, cur, nbits in _helper_cases():
        direct = oracle.apply_quantized(base, cur, nbits)
        via_stream = oracle.recover(base, [oracle.compress(base, cur, nbits)])
        assert np.array_equal(direct.view(np.uint32), via_stream.view(np.uint32))
    base, cur, nbits = _helper_cases()[-2]
    assert oracle.apply_quantized(base, cur, nbits)[:7].view(np.uint32).tolist() == [0] * 7  # -0 + (+0) = +0


def test_compress_chunks_are_slices_of_the_whole_stream(oracle):
    for base, cur, nbits in _helper_cases():
        n = base.size
        s = oracle.compress(base, cur, nbits)
        nchunks = (n + 4095) // 4096
        nsym = int(np.frombuffer(s[16:20].tobytes(), "<u4")[0])
        ci = 64 + 16 * nsym
        li = ci + 8 * (nchunks + 1)
        po = int(np.frombuffer(s[56:64].tobytes(), "<u8")[0])
        chunk_off = np.frombuffer(s[ci:li].tobytes(), "<u8")
        lane_bits = np.frombuffer(s[li:li + 64 * nchunks].tobytes(), "<u2").reshape(nchunks, 32)
        ids = list(range(nchunks))[::-1]  # every chunk, in another order than the stream's
        olane, opay = oracle.compress_chunks(base, cur, nbits, ids)
        for k, c in enumerate(ids):
            assert np.array_equal(olane[k], lane_bits[c])
            assert opay[k].tobytes() == s[po + int(chunk_off[c]): po + int(chunk_off[c + 1])].tobytes()


@pytest.mark.parametrize("threads", [1, 2, 5])
def test_threaded_mode_gives_the_same_bytes(oracle, threads):
    rng = np.random.default_rng(71)
    for n, nbits in ((0, 3), (1, 2), (4096, 4), (9 * 4096 + 123, 5), (70001, 8)):
        base, cur = _random_case(rng, n)
        s = oracle.compress(base, cur, nbits)
        assert oracle.compress(base, cur, nbits, threads=threads).tobytes() == s.tobytes()
        want = oracle.recover(base, [s, s, s])
        got = oracle.recover(base, [s, s, s], threads=threads)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    base = np.linspace(-1, 1, 10000).astype(np.float32)  # a single used symbol: no payload
    s = oracle.compress(base, base, 4, threads=threads)
    assert s.tobytes() == oracle.compress(base, base, 4).tobytes()
    assert np.array_equal(oracle.recover(base, [s], threads=threads).view(np.uint32), (base + np.float32(0)).view(np.uint32))


# ---------------------------------------------------------------- checkpoint merging (Section 3.2)


def test_merge_of_one_stream_over_a_zero_base_is_that_stream(oracle):
    # With base = 0 the recovered state is the quantized delta itself; every kept bucket then holds a single value,
    # its own representative, so quantizing again changes nothing and the merged stream is the stream, byte for byte.
    rng = np.random.default_rng(81)
    for n, nbits in ((10, 2), (5000, 3), (3 * 4096 + 9, 5)):
        cur = rng.laplace(0, 1e-3, n).astype(np.float32)
        base = np.zeros(n, np.float32)
        s = oracle.compress(base, cur, nbits)
        assert oracle.merge(base, [s], nbits).tobytes() == s.tobytes()


def test_merge_is_compress_of_the_recovered_state(oracle):
    rng = np.random.default_rng(82)
    n = 3 * 4096 + 501
    u0 = rng.normal(0, 0.05, n).astype(np.float32)
    u, tracked, streams = u0.copy(), u0.copy(), []
    for t in range(4):
        u = (u + rng.normal(0, 1e-3, n).astype(np.float32)).astype(np.float32)
        s = oracle.compress(tracked, u, 3)
        streams.append(s)
        tracked = oracle.recover(tracked, [s])
    for k in (1, 2, 4):
        m = oracle.merge(u0, streams[:k], 4)
        state_k = oracle.recover(u0, streams[:k])
        assert m.tobytes() == oracle.compress(u0, state_k, 4).tobytes()
        # the super-step checkpoint quantizes a second time: close to the state of the k streams, within the
        # error bound of exponent quantization (half a binade of each kept delta), not identical to it
        back = oracle.recover(u0, [m])
        d = (state_k - u0).astype(np.float32)
        t4 = oracle.table(u0, state_k, 4)
        sym = oracle.symbols(u0, state_k, 4)
        kept = sym > 0
        e = np.floor(np.log2(np.abs(d[kept])))
        assert np.all(np.abs((back - u0)[kept].astype(np.float64) - d[kept]) < 2.0 ** (e - 1) + 2.0 ** -24 * np.abs(u0[kept]) * 2)
        assert np.array_equal(back.view(np.uint32), (u0 + t4["rep"][sym]).view(np.uint32))
    with pytest.raises(oracle.OracleError):
        oracle.merge(u0[:-1], streams[:1], 4)  # element count mismatch


# ---------------------------------------------------------------- fixed-width codes and nbits = 9 (Section 4.3's stages)


def _parse(s):
    nsym = int(np.frombuffer(s[16:20].tobytes(), "<u4")[0])
    n = int(np.frombuffer(s[8:16].tobytes(), "<u8")[0])
    nchunks = (n + 4095) // 4096
    ci = 64 + 16 * nsym
    li = ci + 8 * (nchunks + 1)
    po = int(np.frombuffer(s[56:64].tobytes(), "<u8")[0])
    tab = np.frombuffer(s[64:ci].tobytes(), dtype=[("key", "<u2"), ("len", "u1"), ("pad", "u1"), ("rep", "<u4"), ("count", "<u8")])
    return dict(n=n, nsym=nsym, nchunks=nchunks, tab=tab, chunk_off=np.frombuffer(s[ci:li].tobytes(), "<u8"),
                lane_bits=np.frombuffer(s[li:li + 64 * nchunks].tobytes(), "<u2").reshape(nchunks, 32), po=po,
                payload_bits=int(np.frombuffer(s[40:48].tobytes(), "<u8")[0]), max_len=int(s[20]), flags=int(s[7]),
                nbits=int(s[6]))


def test_paper_example_as_a_fixed_width_stream(oracle):
    # Section 3.1.1's worked example: 10 elements in 5 buckets, every bucket kept (no promotion: nbits 9), fixed
    # 3-bit indices: 10 * 3 bits of payload, and with the 5 representatives of 32 bits each 190 bits, rate 1.68.
    g = load_golden("ten_elements_nbits2.txt")
    base = np.zeros(10, np.float32)
    s = oracle.compress(base, g["cur"], 9, fixed=True)
    p = _parse(s)
    assert p["nbits"] == 9 and p["flags"] == 1
    assert p["nsym"] == 6 and p["max_len"] == 3 and p["payload_bits"] == 30  # 5 buckets + the zero symbol: 3 bits
    assert p["payload_bits"] + 32 * 5 == oracle.model_bits(10, 5, 32) == 190
    assert p["tab"]["len"].tolist() == [3] * 6 and int(p["tab"]["count"][0]) == 0
    # nothing is dropped: every element comes back as its bucket's representative, here the element itself or
    # the midrange of its bucket
    out = oracle.recover(base, [s])
    t = oracle.table(base, g["cur"], 9, fixed=True)
    sym = oracle.symbols(base, g["cur"], 9)
    assert np.all(sym > 0)
    assert np.array_equal(out.view(np.uint32), t["rep"][sym].view(np.uint32))
    # with 2-bit promotion the same vector takes 2 bits per index
    s2 = oracle.compress(base, g["cur"], 2, fixed=True)
    assert _parse(s2)["payload_bits"] == 20 and _parse(s2)["max_len"] == 2


def test_fixed_width_payload_by_independent_bit_writer(oracle):
    rng = np.random.default_rng(91)
    n = 4096 + 777
    base, cur = _random_case(rng, n)
    for nbits in (1, 3, 9):
        s = oracle.compress(base, cur, nbits, fixed=True)
        p = _parse(s)
        sym = oracle.symbols(base, cur, nbits)
        width = max(0, int(p["nsym"] - 1).bit_length())
        assert p["max_len"] == width and p["payload_bits"] == n * width
        assert np.array_equal(oracle.decode_symbols(s, n), sym)
        for c in range(p["nchunks"]):
            bits = ""
            for lane in range(32):
                for j in range(32):
                    for e in range(4):
                        i = 4096 * c + 128 * j + 4 * lane + e
                        if i < n and width:
                            bits += format(int(sym[i]), "0%db" % width)
            nbytes = ((len(bits) + 7) // 8 + 15) // 16 * 16
            bits = bits.ljust(nbytes * 8, "0")
            words = np.array([int(bits[w:w + 32], 2) for w in range(0, len(bits), 32)], "<u4")
            lo = p["po"] + int(p["chunk_off"][c])
            assert s[lo: p["po"] + int(p["chunk_off"][c + 1])].tobytes() == words.tobytes()
        # same symbols and representatives as the Huffman-coded stream: the recovered state is the same
        if nbits <= 8:
            h = oracle.compress(base, cur, nbits)
            assert np.array_equal(oracle.recover(base, [s]).view(np.uint32), oracle.recover(base, [h]).view(np.uint32))
            assert s.size >= h.size - 16 * p["nchunks"]  # Huffman never needs more payload bits than the fixed code


def test_nine_bit_promotion_keeps_every_bucket(oracle):
    # magnitudes over 150 binades, both signs: about 300 occupied buckets, so symbol ids go beyond one byte
    rng = np.random.default_rng(92)
    n = 60000
    cur = (np.exp2(rng.uniform(-100, 50, n)) * rng.choice([-1.0, 1.0], n)).astype(np.float32)
    cur[:100] = 0.0
    base = np.zeros(n, np.float32)
    count, _, _ = oracle.bins(base, cur)
    occupied = int(((count > 0) & (np.arange(512) % 256 >= 1) & (np.arange(512) % 256 <= 254)).sum())
    assert occupied > 255
    for fixed in (False, True):
        s = oracle.compress(base, cur, 9, fixed=fixed)
        p = _parse(s)
        assert p["nsym"] == occupied + 1
        sym = oracle.decode_symbols(s, n)
        assert int(sym.max()) == occupied and np.array_equal(sym, oracle.symbols(base, cur, 9))
        out = oracle.recover(base, [s])
        d = cur
        assert np.all(out[:100] == 0)
        nz = d != 0
        e = np.floor(np.log2(np.abs(d[nz])))
        assert np.all(np.abs(out[nz].astype(np.float64) - d[nz]) < 2.0 ** (e - 1) + 1e-300)  # half a binade at most
    assert oracle.compress(base, cur, 9, fixed=True).tobytes() == oracle.compress(base, cur, 9, fixed=True, threads=3).tobytes()


def test_reader_checks_fixed_width_streams(oracle):
    rng = np.random.default_rng(93)
    base, cur = _random_case(rng, 5000)
    good = oracle.compress(base, cur, 3, fixed=True)
    assert oracle.recover(base, [good]).size == 5000
    bad = good.copy()
    bad[64 + 2] = 2  # one length changed
    huff = oracle.compress(base, cur, 3)
    huff[7] = 1      # a Huffman-coded stream that claims fixed-width codes
    for s in (bad, huff):
        with pytest.raises(oracle.OracleError) as e:
            oracle.recover(base, [s])
        assert e.value.code == oracle.ERR_FORMAT


# ---------------------------------------------------------------- shards of a split vector (format section 1.6)


def test_shards_code_with_the_whole_vectors_table(oracle):
    rng = np.random.default_rng(101)
    n = 5 * 4096 + 321
    base, cur = _random_case(rng, n)
    cur[3 * 4096:] = base[3 * 4096:] + (cur[3 * 4096:] - base[3 * 4096:]) * 64  # the parts differ in scale
    nbits = 3
    whole = oracle.compress(base, cur, nbits)
    pw = _parse(whole)
    sym = oracle.symbols(base, cur, nbits)
    want = oracle.recover(base, [whole])
    cuts = [0, 2 * 4096, 3 * 4096, n]  # chunk-aligned cuts
    counts = np.zeros(pw["nsym"], np.uint64)
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        s = oracle.compress_shard(base, cur, lo, hi, nbits)
        p = _parse(s)
        assert p["flags"] == 2 and p["n"] == hi - lo
        # the same table as the whole vector's, but for the counts, which are the shard's own
        for f in ("key", "len", "rep"):
            assert np.array_equal(p["tab"][f], pw["tab"][f])
        assert np.array_equal(p["tab"]["count"], np.bincount(sym[lo:hi], minlength=pw["nsym"]).astype(np.uint64))
        counts += p["tab"]["count"]
        # its symbols, its chunks and its recovered part are the whole stream's
        assert np.array_equal(oracle.decode_symbols(s, hi - lo), sym[lo:hi])
        c0 = lo // 4096
        for c in range(p["nchunks"]):
            assert np.array_equal(p["lane_bits"][c], pw["lane_bits"][c0 + c])
            a = s[p["po"] + int(p["chunk_off"][c]): p["po"] + int(p["chunk_off"][c + 1])]
            b = whole[pw["po"] + int(pw["chunk_off"][c0 + c]): pw["po"] + int(pw["chunk_off"][c0 + c + 1])]
            assert a.tobytes() == b.tobytes()
        out = oracle.recover(base[lo:hi], [s])
        assert np.array_equal(out.view(np.uint32), want[lo:hi].view(np.uint32))
    assert np.array_equal(counts, pw["tab"]["count"])
    # a single shard that is the whole vector: the whole vector's stream but for the flag
    one = oracle.compress_shard(base, cur, 0, n, nbits)
    one[7] = 0
    assert one.tobytes() == whole.tobytes()
    # a cut inside a chunk: other chunks, the same symbols and state
    s = oracle.compress_shard(base, cur, 1000, 9000, nbits)
    assert np.array_equal(oracle.decode_symbols(s, 8000), sym[1000:9000])
    assert np.array_equal(oracle.recover(base[1000:9000], [s]).view(np.uint32), want[1000:9000].view(np.uint32))
    # the flag is what allows codes for symbols the shard does not use
    unused = oracle.compress_shard(base, cur, 0, 4096, 8)
    if np.any((_parse(unused)["tab"]["count"] == 0) & (_parse(unused)["tab"]["len"] != 0)):
        bad = unused.copy()
        bad[7] = 0
        with pytest.raises(oracle.OracleError):
            oracle.recover(base[:4096], [bad])


# ---- Section 3.2, "Huffman Code Table Caching" (format section 1.7) ------------------------------------------


def test_cached_lengths_hand_worked(oracle):
    cache = oracle.new_cache()
    # first snapshot: five used symbols, nothing cached -> the Huffman lengths, and their sorted list in row 4.
    # The counts are given out of order so that the stored row shows the sort.
    hit, ln = oracle.cached_lengths([1, 8, 2, 4, 1], 3, cache)
    assert not hit and ln.tolist() == [4, 1, 3, 2, 4]
    rows = cache.reshape(512, 512)
    assert rows[4, :6].tolist() == [1, 2, 3, 4, 4, 0] and not rows[:4].any() and not rows[5:].any() and not rows[4, 5:].any()
    # second snapshot, again five used symbols: the cached lengths go to the symbols in the order of their counts,
    # most frequent first. 6+10+12+12+8 = 48 bits <= 20 elements * 3 bits, so the row is used, although the
    # Huffman code of these counts (lengths 3,2,2,3,2) takes 45.
    hit, ln = oracle.cached_lengths([3, 5, 4, 2, 6], 3, cache)
    assert hit and ln.tolist() == [4, 2, 3, 4, 1]
    assert sum(c * int(l) for c, l in zip([3, 5, 4, 2, 6], ln)) == 48
    assert sum(c * int(l) for c, l in zip([3, 5, 4, 2, 6], oracle.huffman([3, 5, 4, 2, 6])[0])) == 45
    assert rows[4, :6].tolist() == [1, 2, 3, 4, 4, 0]  # a hit leaves the row alone
    # equal counts: the smaller symbol id takes the shorter length
    hit, ln = oracle.cached_lengths([5, 5, 5, 5, 2], 3, cache)
    assert hit and ln.tolist() == [1, 2, 3, 4, 4]
    # an unused symbol in between: the row is chosen by the number of USED symbols and the symbol keeps length 0
    hit, ln = oracle.cached_lengths([9, 0, 7, 1, 1, 2], 3, cache)
    assert hit and ln.tolist() == [1, 0, 2, 4, 4, 3]
    # a row that would break the size bound is rebuilt: eight symbols cached from a skewed snapshot, then a
    # uniform one: 10 * (1+2+3+4+5+6+7+7) = 350 bits > 80 * 3
    hit, ln = oracle.cached_lengths([128, 64, 32, 16, 8, 4, 2, 1], 3, cache)
    assert not hit and ln.tolist() == [1, 2, 3, 4, 5, 6, 7, 7] and rows[7, :9].tolist() == [1, 2, 3, 4, 5, 6, 7, 7, 0]
    hit, ln = oracle.cached_lengths([10] * 8, 3, cache)
    assert not hit and ln.tolist() == [3] * 8 and rows[7, :9].tolist() == [3] * 8 + [0]
    # fewer than two used symbols: no code, cache untouched
    before = cache.copy()
    hit, ln = oracle.cached_lengths([0, 7, 0], 2, cache)
    assert not hit and ln.tolist() == [0, 0, 0] and np.array_equal(cache, before)


def test_cached_stream_properties(oracle):
    rng = np.random.default_rng(123)
    n, nbits = 3 * 4096 + 500, 3
    base, cur2 = _random_case(rng, n)  # Laplace deltas: a steep length list
    cur1 = (base + rng.normal(0, 1e-3, n).astype(np.float32)).astype(np.float32)  # Gaussian: same bucket count, flatter
    cache = oracle.new_cache()
    # nothing cached yet: the plain stream, byte for byte, and the row of its used-symbol count gets its lengths
    s1 = oracle.compress_cached(base, cur1, nbits, cache)
    assert s1.tobytes() == oracle.compress(base, cur1, nbits).tobytes()
    p1 = _parse(s1)
    u = int(np.count_nonzero(p1["tab"]["count"]))
    assert u == 8
    rows = cache.reshape(512, 512)
    assert rows[u - 1, :u].tolist() == sorted(p1["tab"]["len"].tolist()) and rows.sum() == rows[u - 1, :u].sum()
    # next snapshot: same number of used symbols -> the cached lengths, handed out by count
    s2 = oracle.compress_cached(base, cur2, nbits, cache)
    plain2 = oracle.compress(base, cur2, nbits)
    p2, q2 = _parse(s2), _parse(plain2)
    assert p2["flags"] == 4 and q2["flags"] == 0
    for f in ("key", "rep", "count"):
        assert np.array_equal(p2["tab"][f], q2["tab"][f])
    order = sorted(range(p2["nsym"]), key=lambda j: (-int(p2["tab"]["count"][j]), j))
    assert [int(p2["tab"]["len"][j]) for j in order] == rows[u - 1, :u].tolist()
    assert p2["payload_bits"] == int(np.sum(p2["tab"]["count"] * p2["tab"]["len"].astype(np.uint64)))
    assert q2["payload_bits"] < p2["payload_bits"] <= n * nbits  # not this snapshot's optimal code, within the bound
    assert sorted(q2["tab"]["len"].tolist()) != rows[u - 1, :u].tolist()
    # the stream is an ordinary stream: same symbols, same recovered state as the plain one
    assert np.array_equal(oracle.decode_symbols(s2, n), oracle.symbols(base, cur2, nbits))
    assert np.array_equal(oracle.recover(base, [s2]).view(np.uint32), oracle.recover(base, [plain2]).view(np.uint32))
    # the cached-lengths flag goes with neither fixed-width codes nor shards
    bad = s2.copy()
    bad[7] = 5
    with pytest.raises(oracle.OracleError):
        oracle.recover(base, [bad])


# ---- variant: bucket mean as the representative (format section 1.8) ------------------------------------------


def _nearest_f32(x):
    """fp32 value nearest to the exact rational x, ties to the even mantissa (by exact comparison of candidates)."""
    from fractions import Fraction

    c = np.float32(float(x))
    cands = {np.float32(c), np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))}
    best = None
    for v in cands:
        dist = abs(Fraction(float(v)) - x)
        even = (int(np.float32(v).view(np.uint32)) & 1) == 0
        key = (dist, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, v)
    return np.float32(best[1])


def test_bucket_mean_hand_cases_and_exact_rational(oracle):
    from fractions import Fraction

    one = np.float32(1.0)
    ulp = np.float32(2.0 ** -23)
    assert oracle.bucket_mean([1.0, 1.25, 1.5]) == np.float32(1.25)
    assert oracle.bucket_mean([one, one + ulp]) == one                           # tie: even mantissa 0
    assert oracle.bucket_mean([one + ulp, one + 2 * ulp]) == one + 2 * ulp       # tie: even mantissa 2
    assert oracle.bucket_mean([one + ulp, one + ulp, one + 2 * ulp]) == one + ulp  # 1 + 4/3 ulp
    assert oracle.bucket_mean([one + ulp, one + 2 * ulp, one + 2 * ulp]) == one + 2 * ulp  # 1 + 5/3 ulp
    assert oracle.bucket_mean([-3.0, -2.0]) == np.float32(-2.5)
    assert oracle.bucket_mean([1.75]) == np.float32(1.75)
    fmax = np.finfo(np.float32).max
    assert oracle.bucket_mean([fmax, fmax, fmax]) == fmax                        # largest binade, no carry
    tiny = np.float32(2.0 ** -126)
    assert oracle.bucket_mean([tiny, tiny * np.float32(1.5)]) == tiny * np.float32(1.25)  # smallest normal binade
    assert np.isnan(oracle.bucket_mean([1.0, 2.0]))                              # not one bucket
    rng = np.random.default_rng(5)
    for _ in range(300):
        e = int(rng.integers(-120, 120))
        k = int(rng.integers(1, 40))
        sig = rng.integers(2 ** 23, 2 ** 24, k)
        if rng.random() < 0.3:
            sig = sig[0] + rng.integers(0, 3, k)  # values a few ulps apart: ties are frequent
            sig = np.minimum(sig, 2 ** 24 - 1)
        sign = -1.0 if rng.random() < 0.5 else 1.0
        vals = (sign * sig.astype(np.float64) * 2.0 ** (e - 23)).astype(np.float32)
        exact = sum(Fraction(float(v)) for v in vals) / k
        assert oracle.bucket_mean(vals) == _nearest_f32(exact)


def test_mean_stream_differs_from_the_plain_one_in_representatives_only(oracle):
    rng = np.random.default_rng(77)
    n, nbits = 2 * 4096 + 300, 3
    base, cur = _random_case(rng, n)
    plain, mean = oracle.compress(base, cur, nbits), oracle.compress_mean(base, cur, nbits)
    p, q = _parse(plain), _parse(mean)
    assert q["flags"] == 8 and p["flags"] == 0
    for f in ("key", "len", "count"):
        assert np.array_equal(p["tab"][f], q["tab"][f])
    same = mean.copy()
    same[7] = 0
    same[64:64 + 16 * q["nsym"]] = plain[64:64 + 16 * p["nsym"]]
    assert same.tobytes() == plain.tobytes()  # header flag and table apart, the same bytes
    # every representative is the rounded exact mean of its bucket's deltas
    d = (cur - base).astype(np.float32)
    sym = oracle.symbols(base, cur, nbits)
    reps = q["tab"]["rep"].view(np.float32)
    from fractions import Fraction

    for j in range(1, q["nsym"]):
        vals = d[sym == j]
        assert vals.size == int(q["tab"]["count"][j])
        assert reps[j] == _nearest_f32(sum(Fraction(float(v)) for v in vals) / vals.size)
    assert reps[0] == 0
    # recovery adds those representatives; the squared error inside the kept buckets is not above the midrange's
    out_mean, out_plain = oracle.recover(base, [mean]), oracle.recover(base, [plain])
    assert np.array_equal(out_mean.view(np.uint32), (base + reps[sym]).astype(np.float32).view(np.uint32))
    kept = sym > 0
    err_mean = np.sum((out_mean.astype(np.float64) - cur)[kept] ** 2)
    err_plain = np.sum((out_plain.astype(np.float64) - cur)[kept] ** 2)
    assert err_mean <= err_plain * (1 + 1e-6)
    # the flag goes alone
    bad = mean.copy()
    bad[7] = 9
    with pytest.raises(oracle.OracleError):
        oracle.recover(base, [bad])
