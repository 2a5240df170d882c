"""The pins are sharp: a plausible mistake planted in a copy of the oracle (on the CPU) makes some pin fail.

Each mutation edits one line of a temporary copy of ``oracle/lc_oracle.cpp``, builds it with g++ and runs a
compact set of pin checks against it. The real oracle must pass the same checks. Nothing here touches the
CUDA path or a GPU.
"""
import ctypes as C
import itertools
import os
import subprocess
import tempfile

import numpy as np
import pytest

from conftest import ROOT, load_golden

SRC = os.path.join(ROOT, "oracle", "lc_oracle.cpp")

MUTATIONS = [
    ("delta sign", "const float d = cur[i] - base[i];", "const float d = base[i] - cur[i];"),
    ("exponent mask", "const int E = static_cast<int>((u >> 23) & 255u);", "const int E = static_cast<int>((u >> 23) & 127u);"),
    ("sign ignored in key", "return 256 * s + E;", "return E;"),
    ("min never updated", "if (d < b.vmin) b.vmin = d;", "if (d > b.vmin) b.vmin = d;"),
    ("selection ascending", "for (int E = 254; E >= 1; --E) {", "for (int E = 1; E <= 254; ++E) {"),
    ("negative before positive", "for (int s = 0; s <= 1; ++s) {\n      const int key = 256 * s + E;\n      if (buckets[key].count > 0 && kept < keep_max)",
     "for (int s = 1; s >= 0; --s) {\n      const int key = 256 * s + E;\n      if (buckets[key].count > 0 && kept < keep_max)"),
    ("keeps 2^x buckets", "const int keep_max = (1 << nbits) - 1;", "const int keep_max = (1 << nbits);"),
    ("mean of min and max dropped", "(static_cast<double>(vmin) + static_cast<double>(vmax)) * 0.5", "static_cast<double>(vmax)"),
    ("midrange in float", "const double mid = (static_cast<double>(vmin) + static_cast<double>(vmax)) * 0.5;",
     "const double mid = static_cast<double>((vmin + vmax) * 0.5f);"),
    ("huffman tie: internal first", "nodes[front_a].weight <= nodes[front_b].weight", "nodes[front_a].weight < nodes[front_b].weight"),
    ("huffman takes largest", "if (count[a] != count[b]) return count[a] < count[b];", "if (count[a] != count[b]) return count[a] > count[b];"),
    ("canonical step", "if (r > 0) next = (next + 1) << (len[j] - prev_len);", "if (r > 0) next = (next << (len[j] - prev_len)) + 1;"),
    ("zero count", "t->count[0] = n - kept_total;", "t->count[0] = n;"),
    ("lane interleave", "return kChunkElems * c + kLanes * kGroup * j + kGroup * lane + e;", "return kChunkElems * c + kSteps * kGroup * lane + kGroup * j + e;"),
    ("bit order in word", "const int pos = 31 - static_cast<int>(b & 31);\n  chunk[4 * word + pos / 8] |=", "const int pos = static_cast<int>(b & 31);\n  chunk[4 * word + pos / 8] |="),
    ("lsb-first codes", "for (int b = t.len[symbol] - 1; b >= 0; --b) {\n          if ((t.code[symbol] >> b) & 1) set_chunk_bit(chunk, bit);",
     "for (int b = 0; b < t.len[symbol]; ++b) {\n          if ((t.code[symbol] >> b) & 1) set_chunk_bit(chunk, bit);"),
    ("chunk not padded to 16", "const uint64_t chunk_bytes = align16((chunk_bits + 7) / 8);", "const uint64_t chunk_bytes = (chunk_bits + 7) / 8;"),
    ("recover subtracts", "x[i] = x[i] + parsed[j].table.rep[sym[i]];", "x[i] = x[i] - parsed[j].table.rep[sym[i]];"),
    ("zero representative not added", "for (uint64_t i = 0; i < n; ++i) x[i] = x[i] + parsed[j].table.rep[sym[i]];",
     "for (uint64_t i = 0; i < n; ++i) if (parsed[j].table.rep[sym[i]] != 0.0f) x[i] = x[i] + parsed[j].table.rep[sym[i]];"),
    ("step 7 helper subtracts", "out[i] = base[i] + t.rep[sel.symbol_of_key[bucket_key(cur[i] - base[i])]];",
     "out[i] = base[i] - t.rep[sel.symbol_of_key[bucket_key(cur[i] - base[i])]];"),
    ("step 7 helper: operands of the delta swapped", "out[i] = base[i] + t.rep[sel.symbol_of_key[bucket_key(cur[i] - base[i])]];",
     "out[i] = base[i] + t.rep[sel.symbol_of_key[bucket_key(base[i] - cur[i])]];"),
    ("chunk helper codes another chunk", "encode_chunk(base, cur, n, t, sel, chunk_ids[k], li, chunk.data(), &bits);",
     "encode_chunk(base, cur, n, t, sel, k, li, chunk.data(), &bits);"),
    ("chunk helper: lane order", "lane_bits[32 * k + lane] = static_cast<uint16_t>(get_le(li + 2 * lane, 2));",
     "lane_bits[32 * k + lane] = static_cast<uint16_t>(get_le(li + 2 * (31 - lane), 2));"),
    ("merge: operands swapped", "return lco_compress(base, recovered.data(), n, nbits, stream, capacity, out_bytes);",
     "return lco_compress(recovered.data(), base, n, nbits, stream, capacity, out_bytes);"),
    ("merge: recovers from zero instead of base", "const int rc = lco_recover(base, streams, stream_bytes, k, n, recovered.data());\n  if (rc != LCO_OK) return rc;\n  return lco_compress",
     "std::vector<float> zero(n, 0.0f);\n  const int rc = lco_recover(zero.data(), streams, stream_bytes, k, n, recovered.data());\n  if (rc != LCO_OK) return rc;\n  return lco_compress"),
    ("threaded statistics: minimum not merged", "if (b.vmin < m.vmin) m.vmin = b.vmin;", "if (b.vmin > m.vmin) m.vmin = b.vmin;"),
    ("threaded recovery: chunk range off by one", "const uint64_t lo = c * kChunkElems, hi = std::min(n, lo + kChunkElems);\n        if (parsed[j].table.max_len == 0)",
     "const uint64_t lo = c * kChunkElems, hi = std::min(n, lo + kChunkElems - 1);\n        if (parsed[j].table.max_len == 0)"),
    ("fixed width one bit short", "while ((1 << width) < t->nsym) width += 1;", "while ((2 << width) < t->nsym) width += 1;"),
    ("fixed-width code is not the symbol id", "t->code[j] = static_cast<uint64_t>(j);", "t->code[j] = static_cast<uint64_t>(t->nsym - 1 - j);"),
    ("shard codes from the vector's first element", "payload_bytes += encode_chunk(base + lo, cur + lo, n, t, sel, c,", "payload_bytes += encode_chunk(base, cur, n, t, sel, c,"),
    ("shard's table built from the shard alone", "delta_buckets(base, cur, n_total, buckets.data());\n  Table t;\n  Selection sel;\n  const int rc = build_table(buckets.data(), n_total, nbits, &t, &sel);\n  if (rc != LCO_OK) return rc;\n  t.shared = 1;",
     "delta_buckets(base + lo, cur + lo, hi - lo, buckets.data());\n  Table t;\n  Selection sel;\n  const int rc = build_table(buckets.data(), hi - lo, nbits, &t, &sel);\n  if (rc != LCO_OK) return rc;\n  t.shared = 1;"),
    ("cache: least frequent symbol gets the shortest length", "if (count[a] != count[b]) return count[a] > count[b];", "if (count[a] != count[b]) return count[a] < count[b];"),
    ("cache: size bound not checked", "if (bits <= static_cast<unsigned __int128>(n) * static_cast<unsigned>(nbits)) {", "if (bits > 0) {"),
    ("cache: row chosen by the table size", "uint8_t* row = cache + static_cast<size_t>(kCacheRowBytes) * (u - 1);", "uint8_t* row = cache + static_cast<size_t>(kCacheRowBytes) * (nsym - 1);"),
    ("cache: row stored unsorted", "std::sort(sorted.begin(), sorted.end());", ""),
    ("cache: a hit is coded with the Huffman lengths", "if (cache) t->cached = cached_lengths(t->count, t->nsym, nbits, n, cache, t->len);\n    else huffman_lengths(t->count, t->nsym, t->len);",
     "if (cache) { std::vector<int> tmp(512); t->cached = cached_lengths(t->count, t->nsym, nbits, n, cache, tmp.data()); }\n    huffman_lengths(t->count, t->nsym, t->len);"),
    ("mean: always rounds down", "if (2 * r > count || (2 * r == count && (sig & 1u))) sig += 1;", ""),
    ("mean: ties away from zero", "(2 * r == count && (sig & 1u))", "(2 * r == count)"),
    ("mean: implicit leading bit dropped", "b.sig_sum += (float_bits(d) & 0x7FFFFFu) | 0x800000u;", "b.sig_sum += (float_bits(d) & 0x7FFFFFu);"),
    ("mean: sign dropped", "return static_cast<float>((key >> 8) ? -magnitude : magnitude);", "return static_cast<float>(magnitude);"),
    ("mean mode still takes the midrange", "t->rep[j] = mean ? bucket_mean(sel.key_of_symbol[j], b.sig_sum, b.count) : midrange(b.vmin, b.vmax);",
     "t->rep[j] = midrange(b.vmin, b.vmax);"),
    ("size model uses floor log", "while ((1ull << width) < k) width += 1;", "while ((2ull << width) <= k) width += 1;"),
]


def _build(text, workdir, name):
    src = os.path.join(workdir, name + ".cpp")
    lib = os.path.join(workdir, name + ".so")
    with open(src, "w") as f:
        f.write(text)
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-ffp-contract=off", "-fPIC", "-shared", "-o", lib, src])
    return lib


class _Oracle:
    """Minimal binding of one oracle build (enough for the checks below)."""

    def __init__(self, path):
        L = C.CDLL(path)
        u64, i32, vp = C.c_uint64, C.c_int, C.c_void_p
        L.lco_huffman.argtypes = [vp, i32, vp, vp]
        L.lco_model_bits.argtypes = [u64, u64, u64]
        L.lco_model_bits.restype = u64
        L.lco_stream_bound.argtypes = [u64, i32]
        L.lco_stream_bound.restype = u64
        L.lco_compress.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_recover.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, vp]
        L.lco_midrange.argtypes = [C.c_float, C.c_float]
        L.lco_midrange.restype = C.c_float
        L.lco_compress_mode.argtypes = [vp, vp, u64, i32, i32, vp, u64, C.POINTER(u64)]
        L.lco_compress_shard.argtypes = [vp, vp, u64, u64, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_compress_cached.argtypes = [vp, vp, u64, i32, vp, vp, u64, C.POINTER(u64)]
        L.lco_cached_lengths.argtypes = [vp, i32, i32, u64, vp, vp]
        L.lco_apply_quantized.argtypes = [vp, vp, u64, i32, vp]
        L.lco_compress_mean.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_bucket_mean.argtypes = [vp, u64]
        L.lco_bucket_mean.restype = C.c_float
        L.lco_compress_chunks.argtypes = [vp, vp, u64, i32, vp, u64, vp, vp, u64, vp]
        L.lco_merge.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_compress_mt.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64), i32]
        L.lco_recover_mt.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, vp, i32]
        self.L = L

    def compress_fixed(self, base, cur, nbits):
        cap = int(self.L.lco_stream_bound(base.size, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        assert self.L.lco_compress_mode(base.ctypes.data, cur.ctypes.data, base.size, nbits, 1, buf.ctypes.data, cap,
                                        C.byref(out)) == 0
        return buf[: out.value].copy()

    def cached_lengths(self, counts, nbits, cache):
        c = np.asarray(counts, np.uint64)
        ln = np.zeros(c.size, np.int32)
        hit = self.L.lco_cached_lengths(c.ctypes.data, c.size, nbits, int(c.sum()), cache.ctypes.data, ln.ctypes.data)
        return bool(hit), ln.tolist()

    def compress_cached(self, base, cur, nbits, cache):
        cap = int(self.L.lco_stream_bound(base.size, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        assert self.L.lco_compress_cached(base.ctypes.data, cur.ctypes.data, base.size, nbits, cache.ctypes.data,
                                          buf.ctypes.data, cap, C.byref(out)) == 0
        return buf[: out.value].copy()

    def bucket_mean(self, values):
        v = np.ascontiguousarray(values, dtype=np.float32)
        return np.float32(self.L.lco_bucket_mean(v.ctypes.data, v.size))

    def compress_mean(self, base, cur, nbits):
        cap = int(self.L.lco_stream_bound(base.size, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        assert self.L.lco_compress_mean(base.ctypes.data, cur.ctypes.data, base.size, nbits, buf.ctypes.data, cap,
                                        C.byref(out)) == 0
        return buf[: out.value].copy()

    def compress_shard(self, base, cur, lo, hi, nbits):
        cap = int(self.L.lco_stream_bound(hi - lo, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        assert self.L.lco_compress_shard(base.ctypes.data, cur.ctypes.data, base.size, lo, hi, nbits, buf.ctypes.data, cap,
                                         C.byref(out)) == 0
        return buf[: out.value].copy()

    def apply_quantized(self, base, cur, nbits):
        out = np.zeros(base.size, np.float32)
        assert self.L.lco_apply_quantized(base.ctypes.data, cur.ctypes.data, base.size, nbits, out.ctypes.data) == 0
        return out

    def compress_chunks(self, base, cur, nbits, ids):
        ids = np.asarray(ids, np.uint64)
        stride = 4096 * 8 + 16
        lane_bits = np.zeros((ids.size, 32), np.uint16)
        payload = np.zeros(ids.size * stride, np.uint8)
        sizes = np.zeros(ids.size, np.uint64)
        assert self.L.lco_compress_chunks(base.ctypes.data, cur.ctypes.data, base.size, nbits, ids.ctypes.data, ids.size,
                                          lane_bits.ctypes.data, payload.ctypes.data, stride, sizes.ctypes.data) == 0
        return lane_bits, [payload[k * stride: k * stride + int(sizes[k])] for k in range(ids.size)]

    def merge(self, base, streams, nbits):
        k = len(streams)
        ptrs = (C.c_void_p * k)(*[s.ctypes.data for s in streams])
        sizes = (C.c_uint64 * k)(*[s.size for s in streams])
        cap = int(self.L.lco_stream_bound(base.size, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        assert self.L.lco_merge(base.ctypes.data, ptrs, sizes, k, base.size, nbits, buf.ctypes.data, cap, C.byref(out)) == 0
        return buf[: out.value].copy()

    def compress_mt(self, base, cur, nbits, threads):
        cap = int(self.L.lco_stream_bound(base.size, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        assert self.L.lco_compress_mt(base.ctypes.data, cur.ctypes.data, base.size, nbits, buf.ctypes.data, cap,
                                      C.byref(out), threads) == 0
        return buf[: out.value].copy()

    def recover_mt(self, base, streams, threads):
        k = len(streams)
        ptrs = (C.c_void_p * k)(*[s.ctypes.data for s in streams])
        sizes = (C.c_uint64 * k)(*[s.size for s in streams])
        out = np.zeros(base.size, np.float32)
        assert self.L.lco_recover_mt(base.ctypes.data, ptrs, sizes, k, base.size, out.ctypes.data, threads) == 0
        return out

    def compress(self, base, cur, nbits):
        cap = int(self.L.lco_stream_bound(base.size, nbits))
        buf = np.zeros(cap + 64, np.uint8)
        out = C.c_uint64(0)
        rc = self.L.lco_compress(base.ctypes.data, cur.ctypes.data, base.size, nbits, buf.ctypes.data, cap, C.byref(out))
        assert rc == 0
        return buf[: out.value].copy()

    def recover(self, base, streams):
        k = len(streams)
        ptrs = (C.c_void_p * k)(*[s.ctypes.data for s in streams])
        sizes = (C.c_uint64 * k)(*[s.size for s in streams])
        out = np.zeros(base.size, np.float32)
        rc = self.L.lco_recover(base.ctypes.data, ptrs, sizes, k, base.size, out.ctypes.data)
        assert rc == 0
        return out

    def huffman(self, counts):
        c = np.asarray(counts, np.uint64)
        ln = np.zeros(c.size, np.int32)
        code = np.zeros(c.size, np.uint64)
        assert self.L.lco_huffman(c.ctypes.data, c.size, ln.ctypes.data, code.ctypes.data) == 0
        return ln, code


def _brute_cost(counts):
    best = None
    for lens in itertools.product(range(1, len(counts) + 1), repeat=len(counts)):
        if sum(2.0 ** -l for l in lens) <= 1.0 + 1e-12:
            cost = sum(c * l for c, l in zip(counts, lens))
            best = cost if best is None else min(best, cost)
    return best


def _pins_hold(o):
    """A compact subset of the pins of test_oracle_pins.py; True if all hold."""
    try:
        for name in ("ten_elements_nbits2.txt", "skew16_nbits3.txt"):
            g = load_golden(name)
            base = np.zeros(g["cur"].size, np.float32)
            if o.compress(base, g["cur"], g["nbits"]).tobytes() != g["stream"].tobytes():
                return False
            if o.recover(base, [g["stream"]]).view(np.uint32).tolist() != g["recovered"].view(np.uint32).tolist():
                return False
        if int(o.L.lco_model_bits(10, 5, 32)) != 190:
            return False
        for counts in ([1, 1, 1, 1, 1], [5, 1, 1, 2, 9], [3, 3, 2, 2, 1, 1]):
            ln, code = o.huffman(counts)
            if sum(c * int(l) for c, l in zip(counts, ln)) != _brute_cost(counts):
                return False
        ln, code = o.huffman([1, 1, 1, 1, 1])
        if ln.tolist() != [3, 3, 2, 2, 2] or code.tolist() != [6, 7, 0, 1, 2]:
            return False
        # leaf against internal node of equal weight: (a+b)=2 ties with c and then with d, leaves go first,
        # so c+d merge and every length is 2 (taking the node first gives 3,3,2,1 at the same cost)
        if o.huffman([1, 1, 2, 2])[0].tolist() != [2, 2, 2, 2]:
            return False
        # exponent fields above 127 and the largest binade
        big = np.array([8.0, 1.0, 3.0e38, 2.0 ** -125], np.float32)  # exponent fields 130, 127, 253, 2
        s3 = o.compress(np.zeros(4, np.float32), big, 3)
        if o.recover(np.zeros(4, np.float32), [s3]).tolist() != big.tolist():
            return False
        fmax = float(np.finfo(np.float32).max)
        if float(o.L.lco_midrange(fmax, fmax)) != fmax:
            return False
        # adding the +0 representative turns a -0.0 base into +0.0
        nz = np.array([0x80000000, 0x3F800000], np.uint32).view(np.float32)
        s2 = o.compress(nz, nz, 2)
        if o.recover(nz, [s2]).view(np.uint32).tolist() != [0, 0x3F800000]:
            return False
        # odd mantissa sum rounds to even; recovery is a plain fp32 add on a base that needs rounding
        lo, hi = np.array([0x3F800001], np.uint32).view(np.float32)[0], np.array([0x3F800002], np.uint32).view(np.float32)[0]
        if np.float32(o.L.lco_midrange(float(lo), float(hi))).view(np.uint32) != 0x3F800002:
            return False
        rng = np.random.default_rng(7)
        n = 6000
        base = rng.normal(0, 0.02, n).astype(np.float32)
        cur = (base + rng.laplace(0, 1e-3, n).astype(np.float32)).astype(np.float32)
        s = o.compress(base, cur, 3)
        out = o.recover(base, [s, s])
        d = cur - base
        once = o.recover(base, [s])
        dq = once - base
        kept = np.abs(dq) > 0
        if not np.all(np.sign(dq[kept]) == np.sign(d[kept])):
            return False
        if not np.array_equal(out.view(np.uint32), o.recover(once, [s]).view(np.uint32)):
            return False
        big = np.abs(d) >= np.abs(d).max() / 2  # the largest deltas are always kept and land within a binade
        if not np.all(np.abs(dq[big] - d[big]) <= np.abs(d[big]) / 2 + 1e-12):
            return False
        # the helpers of the full-size parity tests: step 7 computed directly, single chunks of a stream
        if not np.array_equal(o.apply_quantized(base, cur, 3).view(np.uint32), once.view(np.uint32)):
            return False
        nsym = int(np.frombuffer(s[16:20].tobytes(), "<u4")[0])
        nchunks = (n + 4095) // 4096
        ci = 64 + 16 * nsym
        li = ci + 8 * (nchunks + 1)
        po = int(np.frombuffer(s[56:64].tobytes(), "<u8")[0])
        off = np.frombuffer(s[ci:li].tobytes(), "<u8")
        lanes = np.frombuffer(s[li:li + 64 * nchunks].tobytes(), "<u2").reshape(nchunks, 32)
        olane, opay = o.compress_chunks(base, cur, 3, [1, 0])
        for k, c in enumerate((1, 0)):
            if not np.array_equal(olane[k], lanes[c]) or opay[k].tobytes() != s[po + int(off[c]): po + int(off[c + 1])].tobytes():
                return False
        # checkpoint merging: over a zero base a single stream merges into itself; in general the merged stream
        # recovers the once-more-quantized change on top of the base
        z = np.zeros(n, np.float32)
        sz = o.compress(z, cur, 3)
        if o.merge(z, [sz], 3).tobytes() != sz.tobytes():
            return False
        m = o.merge(base, [s, s], 3)
        if not np.array_equal(o.recover(base, [m]).view(np.uint32), o.apply_quantized(base, out, 3).view(np.uint32)):
            return False
        # fixed-width codes on the paper's example: 10 elements, 5 buckets, 3-bit indices -> 30 payload bits, first
        # payload word = the ids of the four elements of lane 0, then lane 1, ... most significant bit first
        g = load_golden("ten_elements_nbits2.txt")
        zb = np.zeros(10, np.float32)
        sf = o.compress_fixed(zb, g["cur"], 9)
        if int(np.frombuffer(sf[40:48].tobytes(), "<u8")[0]) != 30 or sf[20] != 3:
            return False
        if o.recover(zb, [sf]).view(np.uint32).tolist() != o.apply_quantized(zb, g["cur"], 9).view(np.uint32).tolist():
            return False
        # the Huffman stream of the same vector tells the symbol of every element; the fixed code of symbol j is j
        pof = int(np.frombuffer(sf[56:64].tobytes(), "<u8")[0])
        word0 = int(np.frombuffer(sf[pof:pof + 4].tobytes(), "<u4")[0])
        cur10 = g["cur"]
        keys = [(int(v.view(np.uint32)) >> 31) * 256 + ((int(v.view(np.uint32)) >> 23) & 255) for v in cur10]
        order = sorted(set(keys), key=lambda k: (-(k % 256), k // 256))
        ids = [order.index(k) + 1 for k in keys]
        want_bits = "".join(format(i, "03b") for i in ids).ljust(32, "0")
        if word0 != int(want_bits, 2):
            return False
        # a shard of the vector, coded with the whole vector's table, recovers its part of what the whole stream recovers
        ss = o.compress_shard(base, cur, 4096, n, 3)
        if not np.array_equal(o.recover(base[4096:], [ss]).view(np.uint32), once[4096:].view(np.uint32)):
            return False
        d2 = cur.copy()
        d2[:3000] = base[:3000] + (cur[:3000] - base[:3000]) * 1024  # the first part now holds all the large deltas
        whole2 = o.recover(base, [o.compress(base, d2, 2)])
        s2b = o.compress_shard(base, d2, 3000, n, 2)
        if not np.array_equal(o.recover(base[3000:], [s2b]).view(np.uint32), whole2[3000:].view(np.uint32)):
            return False
        # code-table caching: hand-worked rows (see test_cached_lengths_hand_worked), then a cached stream
        cache = np.zeros(512 * 512, np.uint8)
        rows = cache.reshape(512, 512)
        if o.cached_lengths([1, 8, 2, 4, 1], 3, cache) != (False, [4, 1, 3, 2, 4]) or rows[4, :6].tolist() != [1, 2, 3, 4, 4, 0]:
            return False
        if o.cached_lengths([3, 5, 4, 2, 6], 3, cache) != (True, [4, 2, 3, 4, 1]):
            return False
        if o.cached_lengths([9, 0, 7, 1, 1, 2], 3, cache) != (True, [1, 0, 2, 4, 4, 3]):
            return False
        o.cached_lengths([128, 64, 32, 16, 8, 4, 2, 1], 3, cache)
        if o.cached_lengths([10] * 8, 3, cache) != (False, [3] * 8) or rows[7, :9].tolist() != [3] * 8 + [0]:
            return False
        cache[:] = 0
        if o.compress_cached(base, cur, 3, cache).tobytes() != s.tobytes():
            return False
        # a Gaussian snapshot fills the row of 8 used symbols with a flatter length list; the Laplace snapshot that
        # follows is then coded with those lengths (more bits than its own Huffman code, same symbols and state)
        cache[:] = 0
        cur_g = (base + rng.normal(0, 1e-3, n).astype(np.float32)).astype(np.float32)
        o.compress_cached(base, cur_g, 3, cache)
        sc = o.compress_cached(base, cur, 3, cache)
        nsb = int(np.frombuffer(sc[16:20].tobytes(), "<u4")[0])
        tab = np.frombuffer(sc[64:64 + 16 * nsb].tobytes(), dtype=[("key", "<u2"), ("len", "u1"), ("pad", "u1"), ("rep", "<u4"), ("count", "<u8")])
        used = int(np.count_nonzero(tab["count"]))
        order = sorted(range(nsb), key=lambda j: (-int(tab["count"][j]), j))[:used]
        if sc[7] != 4 or [int(tab["len"][j]) for j in order] != rows[used - 1, :used].tolist():
            return False
        if int(np.frombuffer(sc[40:48].tobytes(), "<u8")[0]) <= int(np.frombuffer(s[40:48].tobytes(), "<u8")[0]):
            return False
        if not np.array_equal(o.recover(base, [sc]).view(np.uint32), once.view(np.uint32)):
            return False
        # mean representatives: hand cases (a tie to even, a third of an ulp, a negative bucket), then a stream whose
        # representatives are the exact means of the deltas of each symbol
        f1, fu = np.float32(1.0), np.float32(2.0 ** -23)
        if o.bucket_mean([f1 + fu, f1 + 2 * fu]) != f1 + 2 * fu or o.bucket_mean([f1, f1 + fu]) != f1:
            return False
        if o.bucket_mean([f1 + fu, f1 + 2 * fu, f1 + 2 * fu]) != f1 + 2 * fu or o.bucket_mean([-3.0, -2.0]) != np.float32(-2.5):
            return False
        sm = o.compress_mean(base, cur, 3)
        if sm[7] != 8:
            return False
        tabm = np.frombuffer(sm[64:64 + 16 * nsym].tobytes(), dtype=[("key", "<u2"), ("len", "u1"), ("pad", "u1"), ("rep", "<f4"), ("count", "<u8")])
        tabp = np.frombuffer(s[64:64 + 16 * nsym].tobytes(), dtype=[("key", "<u2"), ("len", "u1"), ("pad", "u1"), ("rep", "<f4"), ("count", "<u8")])
        changed = 0
        for j in range(1, nsym):
            dbits = d.astype(np.float32).view(np.uint32)
            dkey = (dbits >> 31) * 256 + ((dbits >> 23) & 255)
            vals = d[dkey == int(tabp["key"][j])].astype(np.float64)  # the deltas of symbol j
            if vals.size != int(tabm["count"][j]) or abs(float(tabm["rep"][j]) - vals.mean()) > 2.0 ** -24 * abs(vals.mean()):
                return False
            changed += int(tabm["rep"][j] != tabp["rep"][j])
        if changed == 0:
            return False
        # the threaded timing mode writes the same bytes and states
        if o.compress_mt(base, cur, 3, 3).tobytes() != s.tobytes():
            return False
        if not np.array_equal(o.recover_mt(base, [s, s], 3).view(np.uint32), out.view(np.uint32)):
            return False
        return True
    except AssertionError:
        return False


@pytest.fixture(scope="module")
def workdir():
    with tempfile.TemporaryDirectory() as d:
        yield d


def test_unmodified_oracle_passes_the_compact_pins(workdir):
    assert _pins_hold(_Oracle(_build(open(SRC).read(), workdir, "clean")))


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(workdir, name, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, "mutation target not found: " + name
    mutated = text.replace(old, new, 1)
    lib = _build(mutated, workdir, "mut_" + "".join(ch if ch.isalnum() else "_" for ch in name))
    assert not _pins_hold(_Oracle(lib)), "no pin noticed: " + name
