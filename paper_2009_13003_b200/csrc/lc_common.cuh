// Shared declarations of the CUDA library: format constants, workspace layout, launcher prototypes.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lc.h"

namespace lc {

// ---- stream format, version 1 (docs/FORMAT.md) -------------------------------------------------
constexpr uint32_t kChunkElems = 4096;  // elements per chunk
constexpr uint32_t kLanes = 32;         // lane sub-streams per chunk (one per warp lane)
constexpr uint32_t kGroup = 4;          // consecutive elements a lane takes per step (one float4)
constexpr uint32_t kSteps = kChunkElems / (kLanes * kGroup);  // 32 steps per chunk
constexpr uint32_t kHeaderBytes = 64;
constexpr uint32_t kTableEntryBytes = 16;
constexpr uint32_t kPayloadAlign = 16;
constexpr uint32_t kKeys = 512;  // 256*sign + exponent field
constexpr int kMaxNbits = 9;     // 9 keeps every occupied bucket (at most 508 of them, plus the zero symbol)
constexpr uint32_t kMaxSymbols = 512;

__host__ __device__ constexpr inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

struct StreamLayout {
  uint64_t nchunks, table_off, chunk_index_off, lane_index_off, payload_off;
};

__host__ __device__ inline StreamLayout stream_layout(uint64_t n, uint32_t nsym) {
  StreamLayout L;
  L.nchunks = (n + kChunkElems - 1) / kChunkElems;
  L.table_off = kHeaderBytes;
  L.chunk_index_off = L.table_off + (uint64_t)kTableEntryBytes * nsym;
  L.lane_index_off = L.chunk_index_off + 8 * (L.nchunks + 1);
  L.payload_off = align_up(L.lane_index_off + 64 * L.nchunks, kPayloadAlign);
  return L;
}

// ---- statistics pass -> encode pass hand-over ("key plane") -----------------------------------
// The statistics kernel leaves one byte per element in the workspace so that the encode pass reads
// 1 byte per element instead of 8: ((exponent field & 127) << 1) | sign (the sign in bit 0, so that the two
// signs of an exponent and 16 neighbouring exponents fall into 32 different banks of a table indexed by
// this byte). That identifies the bucket as
// long as every exponent field is below 128, i.e. every |delta| < 2; if some delta is larger (the
// statistics tell), the encode pass ignores the plane and recomputes the keys from base and cur.
// A *unit* is 1024 consecutive elements = 8 steps of one chunk, handled by one warp iteration:
//   unit u: bytes [1024u, 1024u+1024): byte 512*(r/4) + 16*lane + 4*(r%4) + e
// for step r (0..7) of the unit, lane (0..31) and slot e (0..3), i.e. element 1024u + 128r + 4lane + e.
constexpr uint32_t kUnitElems = 1024;
constexpr uint32_t kUnitsPerChunk = kChunkElems / kUnitElems;

// ---- encode pass ----------------------------------------------------------------------------------
constexpr uint32_t kEncWarps = 8;  // warps per CTA of the encode pass (one chunk per warp at a time)

// Chunk descriptor of the decoupled look-back scan of the encode pass: flag in the top two bits, bytes below.
constexpr uint64_t kTileFlagShift = 62;
constexpr uint64_t kTileInvalid = 0, kTileAggregate = 1, kTilePrefix = 2, kTileAbort = 3;
constexpr uint64_t kTileValueMask = (1ull << kTileFlagShift) - 1;

// Entry of the per-key encode table written by the table kernel.
struct EncEntry {
  uint32_t code_lo;  // low 32 bits of the canonical code
  uint32_t len;      // code length in bits (0..63)
  uint32_t code_hi;  // bits 32.. of the code (non-zero only when len > 32)
  uint32_t sym;      // symbol id
};

// Control block at the start of the workspace. Zeroed at the start of every lc_compress.
struct Control {
  int32_t status;         // first device-detected error, 0 if none
  uint32_t ticket;        // next chunk of the encode pass
  uint32_t nsym;          // written by the table kernel
  uint32_t max_len;       // written by the table kernel
  uint64_t payload_bits;  // written by the table kernel
  uint32_t wide;          // written by the table kernel: some delta has an exponent field >= 128
  uint32_t pad32_;
  uint64_t pad_[28];
  unsigned long long count[kKeys];  // elements per key
  uint32_t inv_min[kKeys];          // max over the bucket of ~bits (zero-initialised running minimum)
  uint32_t max_bits[kKeys];         // max over the bucket of bits
  EncEntry enc[kKeys];
  unsigned long long mant_sum[kKeys];  // mean-representative variant only: sum of the bucket's mantissa fields
};
// The bucket statistics as a shard of a split vector hands them out and takes them back (include/lc.h, lc_shard_*):
// the three arrays of Control, in Control's order, so that one copy moves them.
struct ShardStats {
  unsigned long long count[kKeys];
  uint32_t inv_min[kKeys];
  uint32_t max_bits[kKeys];
};
static_assert(sizeof(ShardStats) == LC_STATS_BYTES, "size promised by the header");
static_assert(sizeof(Control) % 256 == 0, "control block must keep the planes 256-byte aligned");

// lc_recover keeps the decode tables of the (at most four) streams of one launch behind the control block, at an
// offset that does not depend on n: the prepare kernel builds them there once, every CTA of the decode kernel copies
// them into its shared memory.
constexpr uint32_t kDecodeImageBytes = 24 * 1024;  // per stream
constexpr uint32_t kDecodeRegionBytes = 4 * kDecodeImageBytes;

struct WorkspaceLayout {
  uint64_t control_off, decode_off, tiles_off, plane_off, total;
  uint64_t nchunks, nunits;
};

__host__ __device__ constexpr inline WorkspaceLayout workspace_layout(uint64_t n) {
  WorkspaceLayout W{};
  W.nchunks = (n + kChunkElems - 1) / kChunkElems;
  W.nunits = W.nchunks * kUnitsPerChunk;
  W.control_off = 0;
  W.decode_off = sizeof(Control);
  W.tiles_off = W.decode_off + kDecodeRegionBytes;              // one 8-byte descriptor per chunk
  W.plane_off = align_up(W.tiles_off + 8 * W.nchunks, 256);
  W.total = align_up(W.plane_off + W.nchunks * kChunkElems, 256);  // 1 byte per element, whole chunks
  return W;
}

// ---- device helpers ----------------------------------------------------------------------------
__device__ inline void set_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

// ---- per-device launch parameters ---------------------------------------------------------------------
// Occupancy figures, SM counts and the "attributes are set" marks that the launchers cache are properties of a
// device (cudaFuncSetAttribute applies to the current device only), so every such cache is an array indexed by
// the device ordinal. Returns -1 if the ordinal cannot be had or is beyond the arrays.
constexpr int kMaxDevices = 64;
inline int current_device_index() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

// How the encode pass finds the byte offset of a tile of chunks, and the limits of its bounded wait.
struct EncodeOptions {
  bool two_pass_scan = false;     // offsets from a sizes pass and a one-CTA scan: no CTA ever waits for another
  uint32_t spin_limit = 1u << 20; // polls of the look-back before it gives up with LC_ERR_TIMEOUT
  uint32_t ticket_bias = 0;       // added to every tile ticket (test aid: with 1, tile 0 is never coded)
  bool fixed_width = false;       // fixed-width codes (format section 1.5) instead of the Huffman code
  bool mean_rep = false;          // bucket means as representatives (format section 1.8) instead of the midrange
  uint8_t* length_cache = nullptr;  // DEVICE, kLengthCacheBytes: code lengths of earlier calls (format section 1.7)
};

constexpr uint32_t kLengthCacheRow = 512;                            // bytes per row: one row per number of used symbols
constexpr uint64_t kLengthCacheBytes = 512ull * kLengthCacheRow;

// Vectors of at most this many elements (one chunk) take the single-CTA, single-launch compress path. Measured per
// call: 24 us at 64 elements, 30 us at 1000, 45 us at 4096, against 44-48 us for the memset and three launches of the
// general path at any of these sizes; from two chunks on the general path is the faster one.
constexpr uint64_t kSmallMaxElems = kChunkElems;

// ---- launchers (each defined next to its kernel) ---------------------------------------------------
// the whole compress pass of a small vector (0 < n <= kSmallMaxElems) in one launch; tracked_out may be null
cudaError_t launch_small_compress(Control* ctl, const float* base, const float* cur, uint64_t n, int nbits,
                                  uint8_t* stream, float* tracked_out, bool keep_status, cudaStream_t cs);
// mean: also accumulate the mantissa sums the mean-representative variant needs (a slower kernel variant)
cudaError_t launch_stats(const float* base, const float* cur, uint64_t n, Control* ctl, uint8_t* plane,
                         cudaStream_t cs, bool mean = false);
// wide_ok: false if the encode pass will not be able to read base and cur (the table pass then rejects a vector
// with an exponent field >= 128 with LC_ERR_RANGE)
// fixed: fixed-width codes (format section 1.5) instead of the Huffman code
// whole: nullptr, or the statistics of the whole vector of which this call codes a shard (format section 1.6):
//        kept buckets, representatives and code then come from them, the table's counts from ctl's own
cudaError_t launch_table(Control* ctl, uint64_t n, int nbits, uint8_t* stream, bool wide_ok, bool fixed,
                         const ShardStats* whole, uint8_t* length_cache, cudaStream_t cs, bool mean = false);
// tracked_out: nullptr, or where to write base + quantized delta (may be base itself)
cudaError_t launch_encode(Control* ctl, unsigned long long* tiles, const uint8_t* plane, const float* base,
                          const float* cur, uint64_t n, uint8_t* stream, float* tracked_out, const EncodeOptions& opt,
                          cudaStream_t cs);

struct DecodeStreams {
  const uint8_t* ptr[4];
  uint64_t bytes[4];
};
// images: kDecodeRegionBytes of device scratch for the streams' decode tables (built by a first small kernel)
// Decodes the chunks [chunk_begin, chunk_end) only (clipped to the vector's chunks). prepare: build the images first
// (false: an earlier launch for the same streams has left them there).
cudaError_t launch_decode(const float* base, const DecodeStreams& streams, int k, uint64_t n, float* out,
                          int32_t* status, void* images, cudaStream_t cs, uint64_t chunk_begin = 0,
                          uint64_t chunk_end = ~0ull, bool prepare = true);

}  // namespace lc
