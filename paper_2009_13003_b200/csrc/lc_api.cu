// C ABI entry points (declared in include/lc.h): argument checks, workspace carving, launch order.
#include <stddef.h>
#include <string.h>

#include "lc_common.cuh"
#include "../../include/lc_debug.h"

using namespace lc;

namespace {

bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

struct Carved {
  Control* ctl;
  unsigned long long* tiles;
  uint8_t* plane;
};

Carved carve(void* workspace, const WorkspaceLayout& W) {
  uint8_t* w = static_cast<uint8_t*>(workspace);
  Carved c;
  c.ctl = reinterpret_cast<Control*>(w + W.control_off);
  c.tiles = reinterpret_cast<unsigned long long*>(w + W.tiles_off);
  c.plane = w + W.plane_off;
  return c;
}

// lc_compress and lc_compress_update: argument checks, then memset + three kernels on `cs`.
int compress_impl(const float* base, const float* cur, uint64_t n, int nbits, void* stream, uint64_t stream_capacity,
                  float* tracked_out, void* workspace, uint64_t workspace_bytes, const EncodeOptions& opt,
                  cudaStream_t cs, bool keep_status = false) {
  if (nbits < 1 || nbits > kMaxNbits || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!stream || !workspace || (n > 0 && (!base || !cur))) return LC_ERR_ARG;
  if (!aligned(base, 16) || !aligned(cur, 16) || !aligned(stream, 16) || !aligned(workspace, 256))
    return LC_ERR_ARG;
  const WorkspaceLayout W = workspace_layout(n);
  if (workspace_bytes < W.total || stream_capacity < lc_stream_bound(n, nbits)) return LC_ERR_CAPACITY;
  const Carved c = carve(workspace, W);

  // a small vector with the default options: one CTA does everything in one launch (no memset either)
  if (n > 0 && n <= kSmallMaxElems && !opt.two_pass_scan && !opt.fixed_width && !opt.mean_rep && !opt.length_cache &&
      opt.ticket_bias == 0 && opt.spin_limit == EncodeOptions().spin_limit) {
    if (launch_small_compress(c.ctl, base, cur, n, nbits, static_cast<uint8_t*>(stream), tracked_out, keep_status, cs) !=
        cudaSuccess)
      return LC_ERR_CUDA;
    return LC_OK;
  }

  // control block and tile descriptors start at zero (keep_status: all but the status word, which holds the
  // outcome of the pass that produced `cur`; the table pass then leaves the vector alone if it is set)
  const uint64_t skip = keep_status ? sizeof(int32_t) : 0;
  cudaError_t e = cudaMemsetAsync(static_cast<uint8_t*>(workspace) + skip, 0, W.plane_off - skip, cs);
  if (e != cudaSuccess) return LC_ERR_CUDA;
  if ((e = launch_stats(base, cur, n, c.ctl, c.plane, cs, opt.mean_rep)) != cudaSuccess) return LC_ERR_CUDA;
  if ((e = launch_table(c.ctl, n, nbits, static_cast<uint8_t*>(stream), true, opt.fixed_width, nullptr, opt.length_cache, cs,
                        opt.mean_rep)) != cudaSuccess)
    return LC_ERR_CUDA;
  if ((e = launch_encode(c.ctl, c.tiles, c.plane, base, cur, n, static_cast<uint8_t*>(stream), tracked_out, opt,
                         cs)) != cudaSuccess)
    return LC_ERR_CUDA;
  return LC_OK;
}

int check_tracked_out(const float* cur, uint64_t n, float*& tracked_out) {
  if (n > 0 && (!tracked_out || !aligned(tracked_out, 16))) return LC_ERR_ARG;
  if (n > 0 && tracked_out == cur) return LC_ERR_ARG;  // cur is read after parts of tracked_out are written
  if (n == 0) tracked_out = nullptr;
  return LC_OK;
}

}  // namespace

extern "C" {

int lc_version(void) { return 100; }

const char* lc_strerror(int code) {
  switch (code) {
    case LC_OK: return "ok";
    case LC_ERR_ARG: return "invalid argument";
    case LC_ERR_CAPACITY: return "buffer too small";
    case LC_ERR_NONFINITE: return "delta contains Inf or NaN";
    case LC_ERR_FORMAT: return "malformed stream";
    case LC_ERR_MISMATCH: return "element count mismatch";
    case LC_ERR_TIMEOUT: return "device-side wait timed out";
    case LC_ERR_CUDA: return "CUDA runtime error";
    case LC_ERR_RANGE: return "a delta of magnitude 2 or more needs the state that the call has released";
    default: return "unknown status";
  }
}

uint64_t lc_stream_bound(uint64_t n, int nbits) {
  if (nbits < 1 || nbits > kMaxNbits) return 0;
  const StreamLayout L = stream_layout(n, 1u << nbits);
  return L.payload_off + (n * (uint64_t)nbits + 7) / 8 + 16 * L.nchunks;
}

uint64_t lc_workspace_bytes(uint64_t n) { return workspace_layout(n).total; }

int lc_compress(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  return compress_impl(base, cur, n, nbits, stream, stream_capacity, nullptr, workspace, workspace_bytes,
                       EncodeOptions(), cs);
}

int lc_compress_update(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                       uint64_t stream_capacity, float* tracked_out, void* workspace, uint64_t workspace_bytes,
                       lc_cuda_stream_t cs) {
  const int rc = check_tracked_out(cur, n, tracked_out);
  if (rc != LC_OK) return rc;
  return compress_impl(base, cur, n, nbits, stream, stream_capacity, tracked_out, workspace, workspace_bytes,
                       EncodeOptions(), cs);
}

int lc_compress_opt(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                    uint64_t stream_capacity, float* tracked_out, void* workspace, uint64_t workspace_bytes,
                    uint32_t options, lc_cuda_stream_t cs) {
  if (options & ~(uint32_t)(LC_OPT_NO_DEVICE_WAIT | LC_OPT_FIXED_WIDTH | LC_OPT_MEAN_REP)) return LC_ERR_ARG;
  if ((options & LC_OPT_MEAN_REP) && (options & LC_OPT_FIXED_WIDTH)) return LC_ERR_ARG;
  if (tracked_out) {
    const int rc = check_tracked_out(cur, n, tracked_out);
    if (rc != LC_OK) return rc;
  }
  EncodeOptions opt;
  opt.two_pass_scan = (options & LC_OPT_NO_DEVICE_WAIT) != 0;
  opt.fixed_width = (options & LC_OPT_FIXED_WIDTH) != 0;
  opt.mean_rep = (options & LC_OPT_MEAN_REP) != 0;
  return compress_impl(base, cur, n, nbits, stream, stream_capacity, tracked_out, workspace, workspace_bytes, opt, cs);
}

int lc_compress_cached(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                       uint64_t stream_capacity, float* tracked_out, void* workspace, uint64_t workspace_bytes,
                       void* length_cache, lc_cuda_stream_t cs) {
  if (!length_cache || !aligned(length_cache, 16)) return LC_ERR_ARG;
  if (tracked_out) {
    const int rc = check_tracked_out(cur, n, tracked_out);
    if (rc != LC_OK) return rc;
  }
  EncodeOptions opt;
  opt.length_cache = static_cast<uint8_t*>(length_cache);
  return compress_impl(base, cur, n, nbits, stream, stream_capacity, tracked_out, workspace, workspace_bytes, opt, cs);
}

int lc_debug_compress_wait(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                           uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, uint32_t spin_limit,
                           uint32_t first_ticket, lc_cuda_stream_t cs) {
  EncodeOptions opt;
  opt.spin_limit = spin_limit;
  opt.ticket_bias = first_ticket;
  return compress_impl(base, cur, n, nbits, stream, stream_capacity, nullptr, workspace, workspace_bytes, opt, cs);
}

int lc_compress_timed(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                      uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs,
                      float* kernel_ms) {
  if (!kernel_ms) return LC_ERR_ARG;
  if (nbits < 1 || nbits > kMaxNbits || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!stream || !workspace || (n > 0 && (!base || !cur))) return LC_ERR_ARG;
  if (!aligned(base, 16) || !aligned(cur, 16) || !aligned(stream, 16) || !aligned(workspace, 256))
    return LC_ERR_ARG;
  const WorkspaceLayout W = workspace_layout(n);
  if (workspace_bytes < W.total || stream_capacity < lc_stream_bound(n, nbits)) return LC_ERR_CAPACITY;
  const Carved c = carve(workspace, W);
  cudaEvent_t ev[4];
  for (int i = 0; i < 4; ++i)
    if (cudaEventCreate(&ev[i]) != cudaSuccess) return LC_ERR_CUDA;
  bool ok = cudaMemsetAsync(workspace, 0, W.plane_off, cs) == cudaSuccess;
  ok = ok && cudaEventRecord(ev[0], cs) == cudaSuccess;
  ok = ok && launch_stats(base, cur, n, c.ctl, c.plane, cs) == cudaSuccess;
  ok = ok && cudaEventRecord(ev[1], cs) == cudaSuccess;
  ok = ok && launch_table(c.ctl, n, nbits, static_cast<uint8_t*>(stream), true, false, nullptr, nullptr, cs) == cudaSuccess;
  ok = ok && cudaEventRecord(ev[2], cs) == cudaSuccess;
  ok = ok && launch_encode(c.ctl, c.tiles, c.plane, base, cur, n, static_cast<uint8_t*>(stream), nullptr, EncodeOptions(), cs) == cudaSuccess;
  ok = ok && cudaEventRecord(ev[3], cs) == cudaSuccess;
  ok = ok && cudaEventSynchronize(ev[3]) == cudaSuccess;
  for (int i = 0; ok && i < 3; ++i) ok = cudaEventElapsedTime(&kernel_ms[i], ev[i], ev[i + 1]) == cudaSuccess;
  for (int i = 0; i < 4; ++i) cudaEventDestroy(ev[i]);
  return ok ? LC_OK : LC_ERR_CUDA;
}

// lc_recover; reset_status: false when an earlier part of the same call may already have set the status word
static int recover_impl(const float* base, const void* const* streams, const uint64_t* stream_bytes, int k,
                        uint64_t n, float* out, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs,
                        bool reset_status) {
  if (k < 1 || k > LC_MAX_CHAIN || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!streams || !stream_bytes || !workspace || (n > 0 && (!base || !out))) return LC_ERR_ARG;
  if (!aligned(base, 16) || !aligned(out, 16) || !aligned(workspace, 256)) return LC_ERR_ARG;
  for (int j = 0; j < k; ++j)
    if (!streams[j] || !aligned(streams[j], 16)) return LC_ERR_ARG;
  if (workspace_bytes < workspace_layout(0).total) return LC_ERR_CAPACITY;
  Control* ctl = static_cast<Control*>(workspace);
  void* images = static_cast<uint8_t*>(workspace) + workspace_layout(0).decode_off;
  if (reset_status && cudaMemsetAsync(&ctl->status, 0, sizeof(int32_t), cs) != cudaSuccess) return LC_ERR_CUDA;
  // up to four streams per launch; later launches continue in place from `out`.
  const float* src = base;
  for (int first = 0; first < k; first += 4) {
    const int kk = (k - first) < 4 ? (k - first) : 4;
    DecodeStreams ds;
    memset(&ds, 0, sizeof ds);
    for (int j = 0; j < kk; ++j) {
      ds.ptr[j] = static_cast<const uint8_t*>(streams[first + j]);
      ds.bytes[j] = stream_bytes[first + j];
    }
    if (launch_decode(src, ds, kk, n, out, &ctl->status, images, cs) != cudaSuccess) return LC_ERR_CUDA;
    src = out;
  }
  return LC_OK;
}

int lc_recover(const float* base, const void* const* streams, const uint64_t* stream_bytes, int k,
               uint64_t n, float* out, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  return recover_impl(base, streams, stream_bytes, k, n, out, workspace, workspace_bytes, cs, true);
}

// ---- per-layer granularity: one stream per segment of the vector --------------------------------------------

static bool segments_ok(const uint64_t* seg_begin, int nseg) {
  if (!seg_begin || nseg < 1 || nseg > LC_MAX_SEGMENTS || seg_begin[0] != 0) return false;
  for (int i = 0; i < nseg; ++i)
    if (seg_begin[i + 1] < seg_begin[i] || (seg_begin[i + 1] & 3u) != 0 || seg_begin[i + 1] - seg_begin[i] >= (1ull << 32))
      return false;
  return true;
}

uint64_t lc_segments_layout(const uint64_t* seg_begin, int nseg, int nbits, uint64_t* stream_offset) {
  if (!segments_ok(seg_begin, nseg) || nbits < 1 || nbits > kMaxNbits) return 0;
  uint64_t off = 0;
  for (int i = 0; i < nseg; ++i) {
    if (stream_offset) stream_offset[i] = off;
    off += align_up(lc_stream_bound(seg_begin[i + 1] - seg_begin[i], nbits), 256);
  }
  if (stream_offset) stream_offset[nseg] = off;
  return off;
}

int lc_compress_segments(const float* base, const float* cur, const uint64_t* seg_begin, int nseg, int nbits,
                         void* streams, uint64_t streams_capacity, float* tracked_out, void* workspace,
                         uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  if (!segments_ok(seg_begin, nseg) || nbits < 1 || nbits > kMaxNbits || !streams || !aligned(streams, 256))
    return LC_ERR_ARG;
  if (streams_capacity < lc_segments_layout(seg_begin, nseg, nbits, nullptr)) return LC_ERR_CAPACITY;
  uint64_t off = 0;
  for (int i = 0; i < nseg; ++i) {
    const uint64_t lo = seg_begin[i], ni = seg_begin[i + 1] - lo;
    const uint64_t cap = align_up(lc_stream_bound(ni, nbits), 256);
    float* t = tracked_out ? tracked_out + lo : nullptr;
    if (t) {
      const int rc = check_tracked_out(cur + lo, ni, t);
      if (rc != LC_OK) return rc;
    }
    // the status word is cleared before the first segment only: a segment the device rejects makes the table and
    // encode passes of all later ones leave their streams invalid, and the word keeps the first failure
    const int rc = compress_impl(base + lo, cur + lo, ni, nbits, static_cast<uint8_t*>(streams) + off, cap, t, workspace,
                                 workspace_bytes, EncodeOptions(), cs, /*keep_status=*/i > 0);
    if (rc != LC_OK) return rc;
    off += cap;
  }
  return LC_OK;
}

int lc_recover_segments(const float* base, const void* const* streams, int k, const uint64_t* seg_begin, int nseg,
                        int nbits, float* out, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  if (!segments_ok(seg_begin, nseg) || nbits < 1 || nbits > kMaxNbits || k < 1 || k > LC_MAX_CHAIN || !streams)
    return LC_ERR_ARG;
  for (int j = 0; j < k; ++j)
    if (!streams[j] || !aligned(streams[j], 256)) return LC_ERR_ARG;
  uint64_t off = 0;
  for (int i = 0; i < nseg; ++i) {
    const uint64_t lo = seg_begin[i], ni = seg_begin[i + 1] - lo;
    const uint64_t cap = align_up(lc_stream_bound(ni, nbits), 256);
    const void* seg_streams[LC_MAX_CHAIN];
    uint64_t seg_bytes[LC_MAX_CHAIN];
    for (int j = 0; j < k; ++j) {
      seg_streams[j] = static_cast<const uint8_t*>(streams[j]) + off;
      seg_bytes[j] = cap;
    }
    const int rc = recover_impl(base + lo, seg_streams, seg_bytes, k, ni, out + lo, workspace, workspace_bytes, cs,
                                /*reset_status=*/i == 0);
    if (rc != LC_OK) return rc;
    off += cap;
  }
  return LC_OK;
}

int lc_compress_async(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                      uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs_state,
                      lc_cuda_stream_t cs_side, lc_cuda_event_t state_read) {
  if (nbits < 1 || nbits > kMaxNbits || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!stream || !workspace || !state_read || cs_state == cs_side || (n > 0 && (!base || !cur))) return LC_ERR_ARG;
  if (!aligned(base, 16) || !aligned(cur, 16) || !aligned(stream, 16) || !aligned(workspace, 256))
    return LC_ERR_ARG;
  const WorkspaceLayout W = workspace_layout(n);
  if (workspace_bytes < W.total || stream_capacity < lc_stream_bound(n, nbits)) return LC_ERR_CAPACITY;
  const Carved c = carve(workspace, W);
  // on the stream that owns the model state: everything that reads it
  if (cudaMemsetAsync(workspace, 0, W.plane_off, cs_state) != cudaSuccess) return LC_ERR_CUDA;
  if (launch_stats(base, cur, n, c.ctl, c.plane, cs_state) != cudaSuccess) return LC_ERR_CUDA;
  if (cudaEventRecord(state_read, cs_state) != cudaSuccess) return LC_ERR_CUDA;
  // beside whatever cs_state does next: table and encode, which work on the bucket statistics and the key plane
  if (cudaStreamWaitEvent(cs_side, state_read, 0) != cudaSuccess) return LC_ERR_CUDA;
  if (launch_table(c.ctl, n, nbits, static_cast<uint8_t*>(stream), /*wide_ok=*/false, false, nullptr, nullptr, cs_side) != cudaSuccess)
    return LC_ERR_CUDA;
  if (launch_encode(c.ctl, c.tiles, c.plane, nullptr, nullptr, n, static_cast<uint8_t*>(stream), nullptr,
                    EncodeOptions(), cs_side) != cudaSuccess)
    return LC_ERR_CUDA;
  return LC_OK;
}

int lc_shard_stats(const float* base, const float* cur, uint64_t n, void* stats, void* workspace,
                   uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  if (n >= (1ull << 32) || !stats || !workspace || (n > 0 && (!base || !cur))) return LC_ERR_ARG;
  if (!aligned(base, 16) || !aligned(cur, 16) || !aligned(stats, 16) || !aligned(workspace, 256)) return LC_ERR_ARG;
  const WorkspaceLayout W = workspace_layout(n);
  if (workspace_bytes < W.total) return LC_ERR_CAPACITY;
  const Carved c = carve(workspace, W);
  if (cudaMemsetAsync(workspace, 0, W.plane_off, cs) != cudaSuccess) return LC_ERR_CUDA;
  if (launch_stats(base, cur, n, c.ctl, c.plane, cs) != cudaSuccess) return LC_ERR_CUDA;
  // count, inv_min, max_bits: contiguous in the control block, in ShardStats' order
  static_assert(offsetof(Control, inv_min) - offsetof(Control, count) == offsetof(ShardStats, inv_min) &&
                    offsetof(Control, max_bits) - offsetof(Control, count) == offsetof(ShardStats, max_bits),
                "one copy moves the three arrays");
  if (cudaMemcpyAsync(stats, c.ctl->count, sizeof(ShardStats), cudaMemcpyDeviceToDevice, cs) != cudaSuccess)
    return LC_ERR_CUDA;
  return LC_OK;
}

int lc_shard_encode(const float* base, const float* cur, uint64_t n, int nbits, const void* whole_stats, void* stream,
                    uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  if (nbits < 1 || nbits > kMaxNbits || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!stream || !workspace || !whole_stats || (n > 0 && (!base || !cur))) return LC_ERR_ARG;
  if (!aligned(base, 16) || !aligned(cur, 16) || !aligned(stream, 16) || !aligned(whole_stats, 16) ||
      !aligned(workspace, 256))
    return LC_ERR_ARG;
  const WorkspaceLayout W = workspace_layout(n);
  if (workspace_bytes < W.total || stream_capacity < lc_stream_bound(n, nbits)) return LC_ERR_CAPACITY;
  const Carved c = carve(workspace, W);
  if (launch_table(c.ctl, n, nbits, static_cast<uint8_t*>(stream), true, false,
                   static_cast<const ShardStats*>(whole_stats), nullptr, cs) != cudaSuccess)
    return LC_ERR_CUDA;
  if (launch_encode(c.ctl, c.tiles, c.plane, base, cur, n, static_cast<uint8_t*>(stream), nullptr, EncodeOptions(),
                    cs) != cudaSuccess)
    return LC_ERR_CUDA;
  return LC_OK;
}

int lc_merge(const float* base, const void* const* streams, const uint64_t* stream_bytes, int k, uint64_t n,
             int nbits, void* stream, uint64_t stream_capacity, float* scratch, void* workspace,
             uint64_t workspace_bytes, lc_cuda_stream_t cs) {
  if (nbits < 1 || nbits > kMaxNbits) return LC_ERR_ARG;
  if (!stream || !aligned(stream, 16) || (n > 0 && (!scratch || !aligned(scratch, 16) || scratch == base)))
    return LC_ERR_ARG;
  if (workspace_bytes < workspace_layout(n).total || stream_capacity < lc_stream_bound(n, nbits)) return LC_ERR_CAPACITY;
  // the state the k streams recover ...
  int rc = lc_recover(base, streams, stream_bytes, k, n, scratch, workspace, workspace_bytes, cs);
  if (rc != LC_OK) return rc;
  // ... coded against the same base. The compress pass starts by clearing the status word, so a stream that the
  // recovery rejected has to be remembered across it: the encode pass leaves, and the status stays, if the word
  // was already set when the table pass looked (see compress_impl's `keep_status`).
  return compress_impl(base, scratch, n, nbits, stream, stream_capacity, nullptr, workspace, workspace_bytes,
                       EncodeOptions(), cs, /*keep_status=*/true);
}

int lc_stream_info(const void* stream, lc_info* info, lc_cuda_stream_t cs) {
  if (!stream || !info) return LC_ERR_ARG;
  uint8_t h[kHeaderBytes];
  if (cudaMemcpyAsync(h, stream, kHeaderBytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return LC_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return LC_ERR_CUDA;
  auto le = [&](int off, int bytes) {
    uint64_t v = 0;
    for (int b = 0; b < bytes; ++b) v |= (uint64_t)h[off + b] << (8 * b);
    return v;
  };
  memset(info, 0, sizeof *info);
  info->nbits = h[6];
  info->fixed_width = h[7] & 1u;
  info->shard = (h[7] >> 1) & 1u;
  info->cached_lengths = (h[7] >> 2) & 1u;
  info->mean_rep = (h[7] >> 3) & 1u;
  info->n = le(8, 8);
  info->nsym = (uint32_t)le(16, 4);
  info->max_len = (uint32_t)le(20, 4);
  info->nchunks = (uint32_t)le(32, 4);
  info->payload_bits = le(40, 8);
  info->total_bytes = le(48, 8);
  info->payload_offset = le(56, 8);
  info->valid = (h[0] == 'L' && h[1] == 'C' && h[2] == 'C' && h[3] == '1' && le(4, 2) == 1 && (h[7] <= 4 || h[7] == 8) &&
                 le(24, 4) == kChunkElems && le(28, 2) == kLanes && le(30, 2) == kGroup &&
                 le(36, 4) == kPayloadAlign)
                    ? 1
                    : 0;
  return LC_OK;
}

int lc_last_status(const void* workspace, lc_cuda_stream_t cs) {
  if (!workspace) return LC_ERR_ARG;
  int32_t st = 0;
  const Control* ctl = static_cast<const Control*>(workspace);
  if (cudaMemcpyAsync(&st, &ctl->status, sizeof st, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return LC_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return LC_ERR_CUDA;
  return st;
}

// ---- host-buffer variants ------------------------------------------------------------------------

uint64_t lc_host_arena_bytes(uint64_t n, int nbits, int k) {
  if (nbits < 1 || nbits > kMaxNbits || k < 1 || k > LC_MAX_CHAIN) return 0;
  const uint64_t vec = align_up(4 * n, 256);
  const uint64_t str = align_up(lc_stream_bound(n, nbits), 256);
  const uint64_t compress = 2 * vec + str;
  const uint64_t recover = vec + (uint64_t)k * str;
  return lc_workspace_bytes(n) + (compress > recover ? compress : recover);
}

int lc_compress_host(const float* base_host, const float* cur_host, uint64_t n, int nbits, void* stream_host,
                     uint64_t stream_capacity, uint64_t* stream_bytes_out, void* arena, uint64_t arena_bytes,
                     lc_cuda_stream_t cs) {
  if (nbits < 1 || nbits > kMaxNbits || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!stream_host || !stream_bytes_out || !arena || !aligned(arena, 256) || (n > 0 && (!base_host || !cur_host)))
    return LC_ERR_ARG;
  const uint64_t bound = lc_stream_bound(n, nbits);
  if (arena_bytes < lc_host_arena_bytes(n, nbits, 1) || stream_capacity < bound) return LC_ERR_CAPACITY;
  uint8_t* a = static_cast<uint8_t*>(arena);
  const uint64_t ws_bytes = lc_workspace_bytes(n), vec = align_up(4 * n, 256);
  float* d_base = reinterpret_cast<float*>(a + ws_bytes);
  float* d_cur = reinterpret_cast<float*>(a + ws_bytes + vec);
  uint8_t* d_stream = a + ws_bytes + 2 * vec;
  if (n > 0) {
    if (cudaMemcpyAsync(d_base, base_host, 4 * n, cudaMemcpyHostToDevice, cs) != cudaSuccess) return LC_ERR_CUDA;
    if (cudaMemcpyAsync(d_cur, cur_host, 4 * n, cudaMemcpyHostToDevice, cs) != cudaSuccess) return LC_ERR_CUDA;
  }
  int rc = lc_compress(d_base, d_cur, n, nbits, d_stream, bound, a, ws_bytes, cs);
  if (rc != LC_OK) return rc;
  if ((rc = lc_last_status(a, cs)) != LC_OK) return rc;
  lc_info info;
  if ((rc = lc_stream_info(d_stream, &info, cs)) != LC_OK) return rc;
  if (!info.valid || info.total_bytes > stream_capacity) return LC_ERR_FORMAT;
  if (cudaMemcpyAsync(stream_host, d_stream, info.total_bytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
    return LC_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return LC_ERR_CUDA;
  *stream_bytes_out = info.total_bytes;
  return LC_OK;
}

}  // extern "C"

namespace {

// The two copy streams and the events of lc_recover_host's pipeline; created per call, destroyed on every way out.
constexpr int kHostSlices = 8;
struct HostPipeline {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t arrived[kHostSlices] = {}, decoded[kHostSlices] = {};
  bool create() {
    if (cudaStreamCreateWithFlags(&in, cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaStreamCreateWithFlags(&out, cudaStreamNonBlocking) != cudaSuccess) return false;
    for (int i = 0; i < kHostSlices; ++i) {
      if (cudaEventCreateWithFlags(&arrived[i], cudaEventDisableTiming) != cudaSuccess) return false;
      if (cudaEventCreateWithFlags(&decoded[i], cudaEventDisableTiming) != cudaSuccess) return false;
    }
    return true;
  }
  ~HostPipeline() {
    for (int i = 0; i < kHostSlices; ++i) {
      if (arrived[i]) cudaEventDestroy(arrived[i]);
      if (decoded[i]) cudaEventDestroy(decoded[i]);
    }
    if (in) cudaStreamDestroy(in);
    if (out) cudaStreamDestroy(out);
  }
};

}  // namespace

extern "C" int lc_recover_host(const float* base_host, const void* const* streams_host, const uint64_t* stream_bytes,
                               int k, uint64_t n, float* out_host, void* arena, uint64_t arena_bytes,
                               lc_cuda_stream_t cs) {
  if (k < 1 || k > LC_MAX_CHAIN || n >= (1ull << 32)) return LC_ERR_ARG;
  if (!streams_host || !stream_bytes || !arena || !aligned(arena, 256) || (n > 0 && (!base_host || !out_host)))
    return LC_ERR_ARG;
  uint8_t* a = static_cast<uint8_t*>(arena);
  const uint64_t ws_bytes = lc_workspace_bytes(n), vec = align_up(4 * n, 256);
  uint64_t need = ws_bytes + vec;
  for (int j = 0; j < k; ++j) {
    if (!streams_host[j]) return LC_ERR_ARG;
    need += align_up(stream_bytes[j], 256);
  }
  if (arena_bytes < need) return LC_ERR_CAPACITY;
  float* d_x = reinterpret_cast<float*>(a + ws_bytes);
  const void* d_streams[LC_MAX_CHAIN];
  uint64_t off = ws_bytes + vec;
  for (int j = 0; j < k; ++j) {
    if (cudaMemcpyAsync(a + off, streams_host[j], stream_bytes[j], cudaMemcpyHostToDevice, cs) != cudaSuccess)
      return LC_ERR_CUDA;
    d_streams[j] = a + off;
    off += align_up(stream_bytes[j], 256);
  }
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  if (nchunks < 16 * kHostSlices) {
    // a small vector: one copy in, one call, one copy out
    if (n > 0 && cudaMemcpyAsync(d_x, base_host, 4 * n, cudaMemcpyHostToDevice, cs) != cudaSuccess) return LC_ERR_CUDA;
    int rc = lc_recover(d_x, d_streams, stream_bytes, k, n, d_x, a, ws_bytes, cs);
    if (rc != LC_OK) return rc;
    if ((rc = lc_last_status(a, cs)) != LC_OK) return rc;
    if (n > 0 && cudaMemcpyAsync(out_host, d_x, 4 * n, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return LC_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return LC_ERR_CUDA;
    return LC_OK;
  }
  // A large vector goes through in slices of whole chunks, so that the two directions of the link work at the same
  // time: slice i of base comes in on one stream, is recovered in place on `cs` as soon as it has arrived (the
  // chunks of a stream decode independently of one another), and leaves on another stream, while slice i + 1 comes in.
  for (int j = 0; j < k; ++j)
    if (!aligned(d_streams[j], 16)) return LC_ERR_ARG;
  HostPipeline pipe;
  if (!pipe.create()) return LC_ERR_CUDA;
  Control* ctl = reinterpret_cast<Control*>(a);
  void* images = a + workspace_layout(0).decode_off;
  if (cudaMemsetAsync(&ctl->status, 0, sizeof(int32_t), cs) != cudaSuccess) return LC_ERR_CUDA;
  const int groups = (k + 3) / 4;
  for (int i = 0; i < kHostSlices; ++i) {
    const uint64_t c0 = nchunks * i / kHostSlices, c1 = nchunks * (i + 1) / kHostSlices;
    const uint64_t e0 = c0 * kChunkElems, e1 = c1 * kChunkElems < n ? c1 * kChunkElems : n;
    if (cudaMemcpyAsync(d_x + e0, base_host + e0, 4 * (e1 - e0), cudaMemcpyHostToDevice, pipe.in) != cudaSuccess)
      return LC_ERR_CUDA;
    if (cudaEventRecord(pipe.arrived[i], pipe.in) != cudaSuccess) return LC_ERR_CUDA;
    if (cudaStreamWaitEvent(cs, pipe.arrived[i], 0) != cudaSuccess) return LC_ERR_CUDA;
    for (int g = 0; g < groups; ++g) {
      const int first = 4 * g, kk = (k - first) < 4 ? (k - first) : 4;
      DecodeStreams ds;
      memset(&ds, 0, sizeof ds);
      for (int j = 0; j < kk; ++j) {
        ds.ptr[j] = static_cast<const uint8_t*>(d_streams[first + j]);
        ds.bytes[j] = stream_bytes[first + j];
      }
      // the decode tables of a group of four streams are built once if there is one group; two groups share the
      // table area and rebuild theirs for every slice
      const bool prepare = groups > 1 || i == 0;
      if (launch_decode(d_x, ds, kk, n, d_x, &ctl->status, images, cs, c0, c1, prepare) != cudaSuccess) return LC_ERR_CUDA;
    }
    if (cudaEventRecord(pipe.decoded[i], cs) != cudaSuccess) return LC_ERR_CUDA;
    if (cudaStreamWaitEvent(pipe.out, pipe.decoded[i], 0) != cudaSuccess) return LC_ERR_CUDA;
    if (cudaMemcpyAsync(out_host + e0, d_x + e0, 4 * (e1 - e0), cudaMemcpyDeviceToHost, pipe.out) != cudaSuccess)
      return LC_ERR_CUDA;
  }
  if (cudaStreamSynchronize(pipe.out) != cudaSuccess || cudaStreamSynchronize(cs) != cudaSuccess) return LC_ERR_CUDA;
  int32_t st = 0;
  if (cudaMemcpy(&st, &ctl->status, sizeof st, cudaMemcpyDeviceToHost) != cudaSuccess) return LC_ERR_CUDA;
  return st;
}

extern "C" {

// ---- stage dumps -----------------------------------------------------------------------------------

int lc_debug_bins(const void* workspace, uint64_t* count, uint32_t* mmin, uint32_t* mmax, lc_cuda_stream_t cs) {
  if (!workspace || !count || !mmin || !mmax) return LC_ERR_ARG;
  const Control* ctl = static_cast<const Control*>(workspace);
  static_assert(sizeof(unsigned long long) == sizeof(uint64_t), "");
  uint32_t inv[kKeys], mx[kKeys];
  if (cudaMemcpyAsync(count, ctl->count, sizeof ctl->count, cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
      cudaMemcpyAsync(inv, ctl->inv_min, sizeof inv, cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
      cudaMemcpyAsync(mx, ctl->max_bits, sizeof mx, cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
      cudaStreamSynchronize(cs) != cudaSuccess)
    return LC_ERR_CUDA;
  for (uint32_t k = 0; k < kKeys; ++k) {
    mmin[k] = count[k] ? ((~inv[k]) & 0x7FFFFFu) : 0x7FFFFFu;
    mmax[k] = count[k] ? (mx[k] & 0x7FFFFFu) : 0u;
  }
  return LC_OK;
}

int lc_debug_codes(const void* workspace, uint32_t* len, uint64_t* code, lc_cuda_stream_t cs) {
  if (!workspace || !len || !code) return LC_ERR_ARG;
  const Control* ctl = static_cast<const Control*>(workspace);
  EncEntry enc[kKeys];
  if (cudaMemcpyAsync(enc, ctl->enc, sizeof enc, cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
      cudaStreamSynchronize(cs) != cudaSuccess)
    return LC_ERR_CUDA;
  for (uint32_t k = 0; k < kKeys; ++k) {
    len[k] = enc[k].len;
    code[k] = ((uint64_t)enc[k].code_hi << 32) | enc[k].code_lo;
  }
  return LC_OK;
}

}  // extern "C"
