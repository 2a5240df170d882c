"""ctypes binding of the C++ CPU oracle (``lc_oracle.cpp``).

Test infrastructure only: the tests, the smoke check and the benchmark's CPU-baseline leg use it to
check and to time the method as the paper states it. The CUDA library never imports this module.
All arrays are numpy arrays in host memory.
"""
import ctypes as C

import numpy as np

from . import build as _build

OK, ERR_ARG, ERR_CAPACITY, ERR_NONFINITE, ERR_FORMAT, ERR_MISMATCH = 0, -1, -2, -3, -4, -5

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        u64, i32, vp = C.c_uint64, C.c_int, C.c_void_p
        L.lco_bins.argtypes = [vp, vp, u64, vp, vp, vp]
        L.lco_table.argtypes = [vp, vp, u64, i32, vp, vp, vp, vp, vp]
        L.lco_symbols.argtypes = [vp, vp, u64, i32, vp]
        L.lco_huffman.argtypes = [vp, i32, vp, vp]
        L.lco_midrange.argtypes = [C.c_float, C.c_float]
        L.lco_midrange.restype = C.c_float
        L.lco_model_bits.argtypes = [u64, u64, u64]
        L.lco_model_bits.restype = u64
        L.lco_stream_bound.argtypes = [u64, i32]
        L.lco_stream_bound.restype = u64
        L.lco_compress.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_decode_symbols.argtypes = [vp, u64, u64, vp]
        L.lco_recover.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, vp]
        L.lco_apply_quantized.argtypes = [vp, vp, u64, i32, vp]
        L.lco_compress_chunks.argtypes = [vp, vp, u64, i32, vp, u64, vp, vp, u64, vp]
        L.lco_table_mode.argtypes = [vp, vp, u64, i32, i32, vp, vp, vp, vp, vp]
        L.lco_compress_mode.argtypes = [vp, vp, u64, i32, i32, vp, u64, C.POINTER(u64)]
        L.lco_compress_mode_mt.argtypes = [vp, vp, u64, i32, i32, vp, u64, C.POINTER(u64), i32]
        L.lco_compress_cached.argtypes = [vp, vp, u64, i32, vp, vp, u64, C.POINTER(u64)]
        L.lco_cached_lengths.argtypes = [vp, i32, i32, u64, vp, vp]
        L.lco_compress_mean.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_bucket_mean.argtypes = [vp, u64]
        L.lco_bucket_mean.restype = C.c_float
        L.lco_compress_shard.argtypes = [vp, vp, u64, u64, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_merge.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, i32, vp, u64, C.POINTER(u64)]
        L.lco_compress_mt.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64), i32]
        L.lco_recover_mt.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, vp, i32]
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle status %d" % code)
        self.code = code


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data


def bins(base, cur):
    """(count[512] u64, mmin[512] u32, mmax[512] u32) of the delta's (sign, exponent) buckets."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    count = np.zeros(512, np.uint64)
    mmin = np.zeros(512, np.uint32)
    mmax = np.zeros(512, np.uint32)
    lib().lco_bins(pb, pc, base.size, count.ctypes.data, mmin.ctypes.data, mmax.ctypes.data)
    return count, mmin, mmax


def table(base, cur, nbits, fixed=False):
    """dict(key, rep, count, len, code), each of length nsym. ``fixed``: fixed-width codes instead of Huffman."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    key = np.zeros(512, np.int32)
    rep = np.zeros(512, np.float32)
    count = np.zeros(512, np.uint64)
    ln = np.zeros(512, np.int32)
    code = np.zeros(512, np.uint64)
    rc = lib().lco_table_mode(pb, pc, base.size, nbits, int(bool(fixed)), key.ctypes.data, rep.ctypes.data,
                              count.ctypes.data, ln.ctypes.data, code.ctypes.data)
    if rc < 0:
        raise OracleError(rc)
    return dict(key=key[:rc], rep=rep[:rc], count=count[:rc], len=ln[:rc], code=code[:rc])


def symbols(base, cur, nbits):
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    sym = np.zeros(base.size, np.uint16)
    rc = lib().lco_symbols(pb, pc, base.size, nbits, sym.ctypes.data)
    if rc < 0:
        raise OracleError(rc)
    return sym


def huffman(count):
    count = np.ascontiguousarray(count, dtype=np.uint64)
    ln = np.zeros(count.size, np.int32)
    code = np.zeros(count.size, np.uint64)
    rc = lib().lco_huffman(count.ctypes.data, count.size, ln.ctypes.data, code.ctypes.data)
    if rc < 0:
        raise OracleError(rc)
    return ln, code


def midrange(vmin, vmax):
    return np.float32(lib().lco_midrange(float(np.float32(vmin)), float(np.float32(vmax))))


def model_bits(n, k, b=32):
    return int(lib().lco_model_bits(n, k, b))


def stream_bound(n, nbits):
    return int(lib().lco_stream_bound(n, nbits))


def compress(base, cur, nbits, threads=None, fixed=False):
    """Returns the stream as a uint8 numpy array. ``threads``: None for the plain single-threaded pass, else the
    number of host threads of the chunk-parallel timing mode (same bytes). ``fixed``: fixed-width bucket indices
    instead of the Huffman code. ``nbits`` 1...9 (9 keeps every bucket)."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    if not 1 <= nbits <= 9:
        raise OracleError(ERR_ARG)
    cap = stream_bound(base.size, nbits)
    buf = np.zeros(cap, np.uint8)
    out = C.c_uint64(0)
    if threads is None:
        rc = lib().lco_compress_mode(pb, pc, base.size, nbits, int(bool(fixed)), buf.ctypes.data, cap, C.byref(out))
    else:
        rc = lib().lco_compress_mode_mt(pb, pc, base.size, nbits, int(bool(fixed)), buf.ctypes.data, cap,
                                        C.byref(out), int(threads))
    if rc < 0:
        raise OracleError(rc)
    return buf[: out.value].copy()


CACHE_BYTES = 512 * 512


def new_cache():
    """An empty length cache (Section 3.2, "Huffman Code Table Caching"): 512 rows of 512 bytes, all zero."""
    return np.zeros(CACHE_BYTES, np.uint8)


def compress_cached(base, cur, nbits, cache):
    """Compress pass that reads and updates the length cache ``cache`` (uint8[CACHE_BYTES], changed in place)."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    assert cache.dtype == np.uint8 and cache.size == CACHE_BYTES and cache.flags.c_contiguous
    cap = stream_bound(base.size, nbits)
    buf = np.zeros(cap, np.uint8)
    out = C.c_uint64(0)
    rc = lib().lco_compress_cached(pb, pc, base.size, nbits, cache.ctypes.data, buf.ctypes.data, cap, C.byref(out))
    if rc < 0:
        raise OracleError(rc)
    return buf[: out.value].copy()


def cached_lengths(count, nbits, cache):
    """The caching step alone: (hit, code lengths) for symbols with the given counts; ``cache`` changed in place."""
    count = np.ascontiguousarray(count, dtype=np.uint64)
    ln = np.zeros(count.size, np.int32)
    hit = lib().lco_cached_lengths(count.ctypes.data, count.size, nbits, int(count.sum()), cache.ctypes.data,
                                   ln.ctypes.data)
    return bool(hit), ln


def compress_mean(base, cur, nbits):
    """Compress pass with bucket means as representatives (format section 1.8)."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    cap = stream_bound(base.size, nbits)
    buf = np.zeros(cap, np.uint8)
    out = C.c_uint64(0)
    rc = lib().lco_compress_mean(pb, pc, base.size, nbits, buf.ctypes.data, cap, C.byref(out))
    if rc < 0:
        raise OracleError(rc)
    return buf[: out.value].copy()


def bucket_mean(values):
    """Representative of the mean variant for values that share sign and exponent."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    return np.float32(lib().lco_bucket_mean(v.ctypes.data, v.size))


def compress_shard(base, cur, lo, hi, nbits):
    """Stream of the elements [lo, hi) coded with the table of the whole vector (a shard of a split vector)."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    cap = stream_bound(hi - lo, nbits)
    buf = np.zeros(cap, np.uint8)
    out = C.c_uint64(0)
    rc = lib().lco_compress_shard(pb, pc, base.size, lo, hi, nbits, buf.ctypes.data, cap, C.byref(out))
    if rc < 0:
        raise OracleError(rc)
    return buf[: out.value].copy()


def decode_symbols(stream, n):
    stream = np.ascontiguousarray(stream, dtype=np.uint8)
    sym = np.zeros(n, np.uint16)
    rc = lib().lco_decode_symbols(stream.ctypes.data, stream.size, n, sym.ctypes.data)
    if rc < 0:
        raise OracleError(rc)
    return sym


def recover(base, streams, threads=None):
    base, pb = _f32(base)
    streams = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    k = len(streams)
    ptrs = (C.c_void_p * k)(*[s.ctypes.data for s in streams])
    sizes = (C.c_uint64 * k)(*[s.size for s in streams])
    out = np.zeros(base.size, np.float32)
    if threads is None:
        rc = lib().lco_recover(pb, ptrs, sizes, k, base.size, out.ctypes.data)
    else:
        rc = lib().lco_recover_mt(pb, ptrs, sizes, k, base.size, out.ctypes.data, int(threads))
    if rc < 0:
        raise OracleError(rc)
    return out


def merge(base, streams, nbits):
    """The super-step stream of Section 3.2 (checkpoint merging): compress(base, recover(base, streams))."""
    base, pb = _f32(base)
    streams = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    k = len(streams)
    ptrs = (C.c_void_p * k)(*[s.ctypes.data for s in streams])
    sizes = (C.c_uint64 * k)(*[s.size for s in streams])
    if not 1 <= nbits <= 9:
        raise OracleError(ERR_ARG)
    cap = stream_bound(base.size, nbits)
    buf = np.zeros(cap, np.uint8)
    out = C.c_uint64(0)
    rc = lib().lco_merge(pb, ptrs, sizes, k, base.size, nbits, buf.ctypes.data, cap, C.byref(out))
    if rc < 0:
        raise OracleError(rc)
    return buf[: out.value].copy()


def apply_quantized(base, cur, nbits):
    """base + quantized(cur - base), computed directly (Algorithm 1 step 7), no bitstream involved."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    out = np.zeros(base.size, np.float32)
    rc = lib().lco_apply_quantized(pb, pc, base.size, nbits, out.ctypes.data)
    if rc < 0:
        raise OracleError(rc)
    return out


def compress_chunks(base, cur, nbits, chunk_ids):
    """(lane_bits[m,32] u16, [payload bytes of each listed chunk]) of the stream for the whole vector."""
    base, pb = _f32(base)
    cur, pc = _f32(cur)
    ids = np.ascontiguousarray(chunk_ids, dtype=np.uint64)
    m = ids.size
    stride = 4096 * 8 + 16
    lane_bits = np.zeros((m, 32), np.uint16)
    payload = np.zeros(m * stride, np.uint8)
    sizes = np.zeros(m, np.uint64)
    rc = lib().lco_compress_chunks(pb, pc, base.size, nbits, ids.ctypes.data, m, lane_bits.ctypes.data,
                                   payload.ctypes.data, stride, sizes.ctypes.data)
    if rc < 0:
        raise OracleError(rc)
    return lane_bits, [payload[k * stride: k * stride + int(sizes[k])].copy() for k in range(m)]
