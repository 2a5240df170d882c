"""Thin ctypes binding of ``liblc.so`` (the C ABI in ``include/lc.h``).

Argument marshalling only: every step of the compress and recovery passes runs in the CUDA kernels.
PyTorch supplies device memory (tensors) and the current CUDA stream. There is no CPU fallback: if the
library cannot be loaded the import of this module's functions fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

OK, ERR_ARG, ERR_CAPACITY, ERR_NONFINITE, ERR_FORMAT, ERR_MISMATCH, ERR_TIMEOUT, ERR_CUDA, ERR_RANGE = 0, -1, -2, -3, -4, -5, -6, -7, -8
MAX_CHAIN = 8

SYMBOLS = (
    "lc_version", "lc_strerror", "lc_stream_bound", "lc_workspace_bytes", "lc_compress", "lc_compress_update", "lc_compress_timed",
    "lc_recover", "lc_compress_opt", "lc_compress_cached",
    "lc_segments_layout", "lc_compress_segments", "lc_recover_segments", "lc_debug_compress_wait", "lc_merge", "lc_compress_async", "lc_shard_stats", "lc_shard_encode",
    "lc_stream_info", "lc_last_status", "lc_host_arena_bytes", "lc_compress_host", "lc_recover_host",
    "lc_debug_bins", "lc_debug_codes", "lc_compress_noalloc",
)
NOALLOC_MAX_N = 4194304


class LCInfo(C.Structure):
    _fields_ = [
        ("n", C.c_uint64), ("total_bytes", C.c_uint64), ("payload_bits", C.c_uint64),
        ("payload_offset", C.c_uint64), ("nbits", C.c_uint32), ("nsym", C.c_uint32),
        ("max_len", C.c_uint32), ("nchunks", C.c_uint32), ("valid", C.c_int32), ("fixed_width", C.c_uint32), ("shard", C.c_uint32),
        ("cached_lengths", C.c_uint32), ("mean_rep", C.c_uint32),
    ]


class LCError(RuntimeError):
    def __init__(self, code, what=""):
        self.code = code
        super().__init__("%s: %s (%d)" % (what, lib().lc_strerror(code).decode(), code))


_lib = None


def lib():
    """Loads (building first if the shared object is missing or stale and nvcc is present) liblc.so."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    try:
        path = _build.build()
    except Exception as e:  # no nvcc here: use what is in the tree
        if not os.path.exists(path):
            raise RuntimeError("liblc.so is missing and could not be built: %s" % e)
    L = C.CDLL(path)
    u64, i32, vp = C.c_uint64, C.c_int, C.c_void_p
    L.lc_version.restype = i32
    L.lc_strerror.argtypes = [i32]
    L.lc_strerror.restype = C.c_char_p
    L.lc_stream_bound.argtypes = [u64, i32]
    L.lc_stream_bound.restype = u64
    L.lc_workspace_bytes.argtypes = [u64]
    L.lc_workspace_bytes.restype = u64
    L.lc_compress.argtypes = [vp, vp, u64, i32, vp, u64, vp, u64, vp]
    L.lc_compress_update.argtypes = [vp, vp, u64, i32, vp, u64, vp, vp, u64, vp]
    L.lc_compress_opt.argtypes = [vp, vp, u64, i32, vp, u64, vp, vp, u64, C.c_uint32, vp]
    L.lc_compress_cached.argtypes = [vp, vp, u64, i32, vp, u64, vp, vp, u64, vp, vp]
    L.lc_segments_layout.argtypes = [C.POINTER(u64), i32, i32, C.POINTER(u64)]
    L.lc_segments_layout.restype = u64
    L.lc_compress_segments.argtypes = [vp, vp, C.POINTER(u64), i32, i32, vp, u64, vp, vp, u64, vp]
    L.lc_recover_segments.argtypes = [vp, C.POINTER(vp), i32, C.POINTER(u64), i32, i32, vp, vp, u64, vp]
    L.lc_debug_compress_wait.argtypes = [vp, vp, u64, i32, vp, u64, vp, u64, C.c_uint32, C.c_uint32, vp]
    L.lc_compress_timed.argtypes = [vp, vp, u64, i32, vp, u64, vp, u64, vp, C.POINTER(C.c_float)]
    L.lc_recover.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, vp, vp, u64, vp]
    L.lc_compress_async.argtypes = [vp, vp, u64, i32, vp, u64, vp, u64, vp, vp, vp]
    L.lc_shard_stats.argtypes = [vp, vp, u64, vp, vp, u64, vp]
    L.lc_shard_encode.argtypes = [vp, vp, u64, i32, vp, vp, u64, vp, u64, vp]
    L.lc_merge.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, i32, vp, u64, vp, vp, u64, vp]
    L.lc_stream_info.argtypes = [vp, C.POINTER(LCInfo), vp]
    L.lc_last_status.argtypes = [vp, vp]
    L.lc_host_arena_bytes.argtypes = [u64, i32, i32]
    L.lc_host_arena_bytes.restype = u64
    L.lc_compress_host.argtypes = [vp, vp, u64, i32, vp, u64, C.POINTER(u64), vp, u64, vp]
    L.lc_recover_host.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), i32, u64, vp, vp, u64, vp]
    L.lc_compress_noalloc.argtypes = [vp, vp, u64, i32, vp, u64, vp]
    L.lc_debug_bins.argtypes = [vp, vp, vp, vp, vp]
    L.lc_debug_codes.argtypes = [vp, vp, vp]
    _lib = L
    return L


def _cs(device):
    return C.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _check(rc, what):
    if rc != OK:
        raise LCError(rc, what)


def stream_bound(n: int, nbits: int) -> int:
    return int(lib().lc_stream_bound(n, nbits))


def workspace_bytes(n: int) -> int:
    return int(lib().lc_workspace_bytes(n))


def alloc_workspace(n: int, device) -> torch.Tensor:
    return torch.empty(workspace_bytes(n), dtype=torch.uint8, device=device)


def alloc_stream(n: int, nbits: int, device) -> torch.Tensor:
    return torch.empty(stream_bound(n, nbits), dtype=torch.uint8, device=device)


def _f32_cuda(t, name):
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise ValueError("%s must be a contiguous float32 CUDA tensor" % name)
    return t


def compress_async(base, cur, nbits, stream, workspace):
    """Enqueues lc_compress on the current stream; no host synchronisation."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    if base.numel() != cur.numel():
        raise ValueError("base and cur differ in size")
    rc = lib().lc_compress(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(),
                           stream.numel(), workspace.data_ptr(), workspace.numel(), _cs(base.device))
    _check(rc, "lc_compress")


def compress_update_async(base, cur, nbits, stream, tracked_out, workspace):
    """Enqueues lc_compress_update on the current stream: the stream of lc_compress plus the advanced tracked state
    in `tracked_out` (which may be `base`); no host synchronisation."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur"), _f32_cuda(tracked_out, "tracked_out")
    if base.numel() != cur.numel() or base.numel() != tracked_out.numel():
        raise ValueError("base, cur and tracked_out differ in size")
    rc = lib().lc_compress_update(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(),
                                  stream.numel(), tracked_out.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                  _cs(base.device))
    _check(rc, "lc_compress_update")


OPT_NO_DEVICE_WAIT = 1
OPT_FIXED_WIDTH = 2
OPT_MEAN_REP = 4


def compress_opt_async(base, cur, nbits, stream, workspace, options, tracked_out=None):
    """Enqueues lc_compress_opt (``options``: 0 or OPT_NO_DEVICE_WAIT; ``tracked_out`` as for lc_compress_update)."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    rc = lib().lc_compress_opt(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(), stream.numel(),
                               None if tracked_out is None else tracked_out.data_ptr(), workspace.data_ptr(),
                               workspace.numel(), options, _cs(base.device))
    _check(rc, "lc_compress_opt")


def debug_compress_wait(base, cur, nbits, stream, workspace, spin_limit, first_ticket):
    """lc_debug_compress_wait: lc_compress with the look-back's poll limit and first tile number given."""
    rc = lib().lc_debug_compress_wait(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(),
                                      stream.numel(), workspace.data_ptr(), workspace.numel(), spin_limit,
                                      first_ticket, _cs(base.device))
    _check(rc, "lc_debug_compress_wait")


def compress_timed(base, cur, nbits, stream, workspace):
    """lc_compress with events around its kernels; returns (stats_ms, table_ms, encode_ms)."""
    ms = (C.c_float * 3)()
    rc = lib().lc_compress_timed(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(),
                                 stream.numel(), workspace.data_ptr(), workspace.numel(), _cs(base.device), ms)
    _check(rc, "lc_compress_timed")
    return tuple(float(x) for x in ms)


def last_status(workspace) -> int:
    return int(lib().lc_last_status(workspace.data_ptr(), _cs(workspace.device)))


def stream_info(stream) -> LCInfo:
    info = LCInfo()
    _check(lib().lc_stream_info(stream.data_ptr(), C.byref(info), _cs(stream.device)), "lc_stream_info")
    return info


def compress(base, cur, nbits, stream=None, workspace=None, fixed=False, mean=False):
    """stream <- LC(cur - base). Returns the stream trimmed to its size (a view of ``stream``). ``fixed``: fixed-width
    bucket indices instead of the Huffman code (LC_OPT_FIXED_WIDTH). ``mean``: bucket means as representatives
    (LC_OPT_MEAN_REP)."""
    n = base.numel()
    if stream is None:
        stream = alloc_stream(n, nbits, base.device)
    if workspace is None:
        workspace = alloc_workspace(n, base.device)
    if fixed or mean:
        compress_opt_async(base, cur, nbits, stream, workspace, (OPT_FIXED_WIDTH if fixed else 0) | (OPT_MEAN_REP if mean else 0))
    else:
        compress_async(base, cur, nbits, stream, workspace)
    _check(last_status(workspace), "lc_compress (device)")
    info = stream_info(stream)
    return stream[: info.total_bytes]


LENGTH_CACHE_BYTES = 262144


def alloc_length_cache(device):
    """An empty length cache for compress_cached (Section 3.2, "Huffman Code Table Caching")."""
    return torch.zeros(LENGTH_CACHE_BYTES, dtype=torch.uint8, device=device)


def compress_cached_async(base, cur, nbits, stream, workspace, length_cache, tracked_out=None):
    """lc_compress_cached on the current stream; no synchronisation."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    rc = lib().lc_compress_cached(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(), stream.numel(),
                                  tracked_out.data_ptr() if tracked_out is not None else None, workspace.data_ptr(),
                                  workspace.numel(), length_cache.data_ptr(), _cs(base.device))
    _check(rc, "lc_compress_cached")


def compress_cached(base, cur, nbits, length_cache, stream=None, workspace=None, tracked_out=None):
    """stream <- LC(cur - base), code lengths taken from / stored in ``length_cache`` (changed in place)."""
    n = base.numel()
    if stream is None:
        stream = alloc_stream(n, nbits, base.device)
    if workspace is None:
        workspace = alloc_workspace(n, base.device)
    compress_cached_async(base, cur, nbits, stream, workspace, length_cache, tracked_out)
    _check(last_status(workspace), "lc_compress_cached (device)")
    return stream[: stream_info(stream).total_bytes]


def segments_layout(seg_begin, nbits):
    """(stream offsets, total bytes) of the streams buffer for the segments that start at ``seg_begin`` (nseg + 1
    element offsets)."""
    nseg = len(seg_begin) - 1
    sb = (C.c_uint64 * (nseg + 1))(*seg_begin)
    off = (C.c_uint64 * (nseg + 1))()
    total = int(lib().lc_segments_layout(sb, nseg, nbits, off))
    if total == 0 and nseg > 0:
        raise LCError(ERR_ARG, "lc_segments_layout")
    return [int(x) for x in off], total


def compress_segments_async(base, cur, seg_begin, nbits, streams, workspace, tracked_out=None):
    """lc_compress_segments on the current stream; no synchronisation."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    nseg = len(seg_begin) - 1
    sb = (C.c_uint64 * (nseg + 1))(*seg_begin)
    rc = lib().lc_compress_segments(base.data_ptr(), cur.data_ptr(), sb, nseg, nbits, streams.data_ptr(), streams.numel(),
                                    tracked_out.data_ptr() if tracked_out is not None else None, workspace.data_ptr(),
                                    workspace.numel(), _cs(base.device))
    _check(rc, "lc_compress_segments")


def compress_segments(base, cur, seg_begin, nbits, streams=None, workspace=None, tracked_out=None):
    """One stream per segment. Returns (streams buffer, offsets): segment i's stream starts at offsets[i]."""
    offsets, total = segments_layout(seg_begin, nbits)
    if streams is None:
        streams = torch.empty(total, dtype=torch.uint8, device=base.device)
    if workspace is None:
        longest = max([b - a for a, b in zip(seg_begin[:-1], seg_begin[1:])] + [0])
        workspace = alloc_workspace(longest, base.device)
    compress_segments_async(base, cur, seg_begin, nbits, streams, workspace, tracked_out)
    _check(last_status(workspace), "lc_compress_segments (device)")
    return streams, offsets


def recover_segments_async(base, streams_list, seg_begin, nbits, out, workspace):
    """lc_recover_segments on the current stream; ``streams_list``: the buffers of a chain, in order."""
    nseg, k = len(seg_begin) - 1, len(streams_list)
    sb = (C.c_uint64 * (nseg + 1))(*seg_begin)
    ptrs = (C.c_void_p * k)(*[s.data_ptr() for s in streams_list])
    rc = lib().lc_recover_segments(base.data_ptr(), ptrs, k, sb, nseg, nbits, out.data_ptr(), workspace.data_ptr(),
                                   workspace.numel(), _cs(base.device))
    _check(rc, "lc_recover_segments")


def recover_segments(base, streams_list, seg_begin, nbits, out=None, workspace=None):
    if out is None:
        out = torch.empty_like(base)
    if workspace is None:
        workspace = alloc_workspace(0, base.device)
    recover_segments_async(base, streams_list, seg_begin, nbits, out, workspace)
    _check(last_status(workspace), "lc_recover_segments (device)")
    return out


def compress_update(base, cur, nbits, tracked_out=None, stream=None, workspace=None):
    """stream <- LC(cur - base) and tracked_out <- base + quantized delta in one call (``tracked_out`` may be
    ``base``; allocated if None). Returns (stream trimmed to its size, tracked_out)."""
    n = base.numel()
    if stream is None:
        stream = alloc_stream(n, nbits, base.device)
    if workspace is None:
        workspace = alloc_workspace(n, base.device)
    if tracked_out is None:
        tracked_out = torch.empty_like(base)
    compress_update_async(base, cur, nbits, stream, tracked_out, workspace)
    _check(last_status(workspace), "lc_compress_update (device)")
    info = stream_info(stream)
    return stream[: info.total_bytes], tracked_out


def recover_async(base, streams, out, workspace):
    _f32_cuda(base, "base"), _f32_cuda(out, "out")
    k = len(streams)
    ptrs = (C.c_void_p * k)(*[s.data_ptr() for s in streams])
    sizes = (C.c_uint64 * k)(*[s.numel() for s in streams])
    rc = lib().lc_recover(base.data_ptr(), ptrs, sizes, k, base.numel(), out.data_ptr(), workspace.data_ptr(),
                          workspace.numel(), _cs(base.device))
    _check(rc, "lc_recover")


def recover(base, streams, out=None, workspace=None):
    """out <- base + sum of the deltas decoded from ``streams`` (applied in order)."""
    if out is None:
        out = torch.empty_like(base)
    if workspace is None:
        workspace = alloc_workspace(0, base.device)
    recover_async(base, streams, out, workspace)
    _check(last_status(workspace), "lc_recover (device)")
    return out


def compress_two_streams(base, cur, nbits, stream, workspace, state_stream, side_stream, state_read):
    """Enqueues lc_compress_async: the statistics pass on `state_stream` (torch.cuda.Stream), then `state_read`
    (torch.cuda.Event) recorded there; table and encode on `side_stream` behind that event."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    if not state_read.cuda_event:  # torch creates the CUDA event at its first record
        state_read.record(state_stream)
    rc = lib().lc_compress_async(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(),
                                 stream.numel(), workspace.data_ptr(), workspace.numel(),
                                 C.c_void_p(state_stream.cuda_stream), C.c_void_p(side_stream.cuda_stream),
                                 C.c_void_p(state_read.cuda_event))
    _check(rc, "lc_compress_async")


STATS_BYTES = 8192


def shard_stats(base, cur, workspace, stats=None):
    """lc_shard_stats: the statistics pass of one shard; returns the 8 KB statistics buffer (uint8 tensor)."""
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    if stats is None:
        stats = torch.empty(STATS_BYTES, dtype=torch.uint8, device=base.device)
    _check(lib().lc_shard_stats(base.data_ptr(), cur.data_ptr(), base.numel(), stats.data_ptr(), workspace.data_ptr(),
                                workspace.numel(), _cs(base.device)), "lc_shard_stats")
    return stats


def combine_stats(buffers):
    """Element-wise combination of shards' statistics buffers on one device (what an all-reduce over the shards
    computes): counts add, the two running-maximum arrays take the unsigned maximum."""
    counts = torch.stack([b[:4096].view(torch.int64) for b in buffers]).sum(0)
    # unsigned 32-bit maximum through int64 (the words can have their top bit set)
    words = torch.stack([b[4096:].view(torch.int32).to(torch.int64) & 0xFFFFFFFF for b in buffers]).amax(0)
    out = torch.empty_like(buffers[0])
    out[:4096] = counts.view(torch.uint8)
    out[4096:] = words.to(torch.int32).view(torch.uint8)  # truncation keeps the low 32 bits
    return out


def all_reduce_stats(stats, group=None):
    """The exchange between lc_shard_stats and lc_shard_encode over a torch.distributed group: after it every rank
    holds the statistics of the whole vector. Two small all-reduces (512 sums, 1024 maxima)."""
    import torch.distributed as dist

    counts = stats[:4096].view(torch.int64).clone()
    words = stats[4096:].view(torch.int32).to(torch.int64) & 0xFFFFFFFF  # unsigned values in a signed type
    dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(words, op=dist.ReduceOp.MAX, group=group)
    stats[:4096] = counts.view(torch.uint8)
    stats[4096:] = words.to(torch.int32).view(torch.uint8)  # truncation keeps the low 32 bits
    return stats


def shard_encode(base, cur, nbits, whole_stats, workspace, stream=None):
    """lc_shard_encode: table and encode pass of one shard with the whole vector's statistics; returns the stream."""
    n = base.numel()
    if stream is None:
        stream = alloc_stream(n, nbits, base.device)
    _check(lib().lc_shard_encode(base.data_ptr(), cur.data_ptr(), n, nbits, whole_stats.data_ptr(), stream.data_ptr(),
                                 stream.numel(), workspace.data_ptr(), workspace.numel(), _cs(base.device)),
           "lc_shard_encode")
    _check(last_status(workspace), "lc_shard_encode (device)")
    return stream[: stream_info(stream).total_bytes]


def merge_async(base, streams, nbits, stream, scratch, workspace):
    """Enqueues lc_merge: the super-step stream of `streams` over `base` (Section 3.2, checkpoint merging)."""
    _f32_cuda(base, "base"), _f32_cuda(scratch, "scratch")
    k = len(streams)
    ptrs = (C.c_void_p * k)(*[s.data_ptr() for s in streams])
    sizes = (C.c_uint64 * k)(*[s.numel() for s in streams])
    rc = lib().lc_merge(base.data_ptr(), ptrs, sizes, k, base.numel(), nbits, stream.data_ptr(), stream.numel(),
                        scratch.data_ptr(), workspace.data_ptr(), workspace.numel(), _cs(base.device))
    _check(rc, "lc_merge")


def merge(base, streams, nbits, stream=None, scratch=None, workspace=None):
    """One stream that stands for `streams` applied to `base`: compress(base, recover(base, streams)). Returns the
    merged stream trimmed to its size; `scratch` (allocated if None) receives the recovered state."""
    n = base.numel()
    if stream is None:
        stream = alloc_stream(n, nbits, base.device)
    if scratch is None:
        scratch = torch.empty_like(base)
    if workspace is None:
        workspace = alloc_workspace(n, base.device)
    merge_async(base, streams, nbits, stream, scratch, workspace)
    _check(last_status(workspace), "lc_merge (device)")
    return stream[: stream_info(stream).total_bytes]


def host_arena_bytes(n, nbits, k) -> int:
    return int(lib().lc_host_arena_bytes(n, nbits, k))


def compress_host(base_cpu, cur_cpu, nbits, stream_cpu, arena):
    """Host-buffer compress: copies in, runs, copies the stream out. Returns the stream size."""
    out = C.c_uint64(0)
    rc = lib().lc_compress_host(base_cpu.data_ptr(), cur_cpu.data_ptr(), base_cpu.numel(), nbits,
                                stream_cpu.data_ptr(), stream_cpu.numel(), C.byref(out), arena.data_ptr(),
                                arena.numel(), _cs(arena.device))
    _check(rc, "lc_compress_host")
    return int(out.value)


def recover_host(base_cpu, streams_cpu, out_cpu, arena):
    k = len(streams_cpu)
    ptrs = (C.c_void_p * k)(*[s.data_ptr() for s in streams_cpu])
    sizes = (C.c_uint64 * k)(*[s.numel() for s in streams_cpu])
    rc = lib().lc_recover_host(base_cpu.data_ptr(), ptrs, sizes, k, base_cpu.numel(), out_cpu.data_ptr(),
                               arena.data_ptr(), arena.numel(), _cs(arena.device))
    _check(rc, "lc_recover_host")
    return out_cpu


def debug_bins(workspace):
    import numpy as np

    count = np.zeros(512, np.uint64)
    mmin = np.zeros(512, np.uint32)
    mmax = np.zeros(512, np.uint32)
    _check(lib().lc_debug_bins(workspace.data_ptr(), count.ctypes.data, mmin.ctypes.data, mmax.ctypes.data,
                               _cs(workspace.device)), "lc_debug_bins")
    return count, mmin, mmax


def debug_codes(workspace):
    import numpy as np

    ln = np.zeros(512, np.uint32)
    code = np.zeros(512, np.uint64)
    _check(lib().lc_debug_codes(workspace.data_ptr(), ln.ctypes.data, code.ctypes.data, _cs(workspace.device)),
           "lc_debug_codes")
    return ln, code


def compress_noalloc(base, cur, nbits, stream):
    """lc_compress_noalloc: compress with the library's built-in scratch (n <= NOALLOC_MAX_N).

    For callers that cannot allocate device memory when a snapshot is taken. Waits for the current
    stream; returns the stream trimmed to its size. Calls must not overlap on one GPU.
    """
    _f32_cuda(base, "base"), _f32_cuda(cur, "cur")
    rc = lib().lc_compress_noalloc(base.data_ptr(), cur.data_ptr(), base.numel(), nbits, stream.data_ptr(),
                                   stream.numel(), _cs(base.device))
    _check(rc, "lc_compress_noalloc")
    return stream[: stream_info(stream).total_bytes]
