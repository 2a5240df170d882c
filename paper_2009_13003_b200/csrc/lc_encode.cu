// Encode pass: key plane -> Huffman bitstream with chunk and lane indices.
//
// Paper: Algorithm 1 step 6 and Section 3.1.2 (the quantized delta, i.e. the sequence of bucket
// indices, is Huffman-coded). Element order, bit order and the two indices are those of the stream
// format text, sections 2 and 3.
//
// One warp codes one chunk of 4096 elements; lane t owns lane sub-stream t. Per chunk:
//   A. every lane sums the code lengths of its 128 elements            -> lane index, chunk size
//   B. the chunk's bits are assembled in a warp-private shared-memory staging area (every lane ORs its
//      words in at its bit offset, found with a warp shuffle scan of the lane lengths)
//   C. the chunk's byte offset comes from an exclusive scan over all chunks, done across CTAs with a
//      decoupled look-back over per-tile descriptors (a tile = the 8 chunks of one CTA iteration);
//   D. the staged chunk is copied to the payload with coalesced 16-byte stores.
// Tiles are handed out by an atomic ticket, so every tile a CTA waits for has already been started by
// a running CTA. The wait is bounded all the same: after kSpinLimit polls the CTA records
// LC_ERR_TIMEOUT, marks its tile aborted (successors see that at once and abort too) and moves on.
//
// Bound: reads 1.125 bytes and writes about 0.5 bytes per element, so this pass is limited by the
// integer work per element, not by HBM.
#include "lc_common.cuh"

namespace lc {
namespace {

constexpr int kEncThreads = kEncWarps * 32;
constexpr uint32_t kStageWords = 1536;  // per warp: 6 KB = 12 bits per element on average
constexpr uint32_t kEncSmem = kEncWarps * kStageWords * 4;
constexpr uint32_t kSpinLimit = 1u << 20;

struct Tables {
  uint2 enc[kKeys];       // {code_lo, len}
  uint32_t enc_hi[kKeys];
};

// Index into the encode table of slot e of a row: exponent byte e of `word`, sign from bit (3 - e) of
// the row's sign nibble.
__device__ __forceinline__ uint32_t key_of(uint32_t word, uint32_t nibble, int e) {
  return ((word >> (8 * e)) & 255u) | (((nibble >> (3 - e)) & 1u) << 8);
}

// Appends a code of at most 32 bits to the lane's bit accumulator and emits completed 32-bit words.
struct Packer {
  unsigned long long acc;  // pending bits in the low `nb` bits
  uint32_t nb;
  uint32_t* dst;  // next word of the chunk this lane touches
  __device__ __forceinline__ void put(uint32_t code, uint32_t len) {
    acc = (acc << len) | code;
    nb += len;
    if (nb >= 32) {
      nb -= 32;
      atomicOr(dst, (uint32_t)(acc >> nb));
      dst += 1;
    }
  }
  __device__ __forceinline__ void flush() {
    if (nb > 0) atomicOr(dst, (uint32_t)(acc << (32 - nb)));
  }
};

// Slow, compact path for the three rare cases: the ragged last chunk, codes longer than 32 bits, and
// a chunk too large for the staging area. Reads the plane from global memory element by element.
// With dst == nullptr it only returns the lane's bit count.
__device__ __noinline__ uint32_t chunk_slow(const Tables& tb, const uint8_t* __restrict__ eplane,
                                            const uint32_t* __restrict__ splane, uint64_t c, uint32_t lane,
                                            uint64_t n, uint32_t* dst, uint32_t lane_start) {
  Packer pk{0ull, lane_start & 31u, dst ? dst + (lane_start >> 5) : nullptr};
  uint32_t bits = 0;
  for (uint32_t j = 0; j < kSteps; ++j) {
    const uint32_t sw = splane[c * 128 + (j >> 3) * 32 + lane];
    for (uint32_t e = 0; e < kGroup; ++e) {
      const uint64_t i = c * kChunkElems + 128ull * j + 4 * lane + e;
      if (i >= n) continue;
      const uint32_t E = eplane[c * kChunkElems + (j >> 2) * 512 + lane * 16 + (j & 3) * 4 + e];
      const uint32_t s = (sw >> (31 - ((j & 7) * 4 + e))) & 1u;
      const uint32_t key = E | (s << 8);
      const uint2 en = tb.enc[key];
      bits += en.y;
      if (dst) {
        if (en.y > 32) {
          pk.put(tb.enc_hi[key], en.y - 32);
          pk.put(en.x, 32);
        } else {
          pk.put(en.x, en.y);
        }
      }
    }
  }
  if (dst) pk.flush();
  return bits;
}

__device__ __forceinline__ unsigned long long ld_tile(const unsigned long long* p) {
  return *reinterpret_cast<const volatile unsigned long long*>(p);
}
__device__ __forceinline__ void st_tile(unsigned long long* p, unsigned long long v) {
  *reinterpret_cast<volatile unsigned long long*>(p) = v;
}

__global__ void __launch_bounds__(kEncThreads)
encode_kernel(Control* __restrict__ ctl, unsigned long long* __restrict__ tiles,
              const uint8_t* __restrict__ eplane, const uint32_t* __restrict__ splane, uint64_t n,
              uint8_t* __restrict__ stream) {
  extern __shared__ __align__(16) uint32_t s_stage_all[];
  __shared__ Tables tb;
  __shared__ uint32_t s_chunk_bytes[kEncWarps];
  __shared__ uint32_t s_tile;
  __shared__ unsigned long long s_tile_base;
  __shared__ int s_abort;

  if (ctl->status != 0) return;  // the table pass rejected the vector

  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (uint32_t k = tid; k < kKeys; k += kEncThreads) {
    const EncEntry e = ctl->enc[k];
    tb.enc[k] = make_uint2(e.code_lo, e.len);
    tb.enc_hi[k] = e.code_hi;
  }
  const uint32_t nsym = ctl->nsym;
  const bool long_codes = ctl->max_len > 32;
  const StreamLayout L = stream_layout(n, nsym);
  const uint64_t nchunks = L.nchunks;
  const uint64_t ntiles = (nchunks + kEncWarps - 1) / kEncWarps;
  unsigned long long* chunk_index = reinterpret_cast<unsigned long long*>(stream + L.chunk_index_off);
  uint16_t* lane_index = reinterpret_cast<uint16_t*>(stream + L.lane_index_off);
  uint8_t* payload = stream + L.payload_off;
  uint32_t* stage = s_stage_all + warp * kStageWords;

  while (true) {
    __syncthreads();  // previous iteration is done with s_tile, s_chunk_bytes and the staging areas
    if (tid == 0) {
      s_tile = atomicAdd(&ctl->ticket, 1u);
      s_abort = 0;
    }
    __syncthreads();
    const uint64_t tile = s_tile;
    if (tile >= ntiles) break;
    const uint64_t c = tile * kEncWarps + warp;
    const bool valid = c < nchunks;
    const bool full = valid && (c + 1) * kChunkElems <= n;
    const bool fast = full && !long_codes;

    // ---- load the chunk's slice of the key plane: 128 exponent bytes and 128 sign bits per lane
    uint4 ev[8];
    uint32_t sg[4];
    if (fast) {
      const uint4* ep = reinterpret_cast<const uint4*>(eplane + c * kChunkElems) + lane;
#pragma unroll
      for (int q = 0; q < 8; ++q) ev[q] = __ldg(ep + 32 * q);
#pragma unroll
      for (int g = 0; g < 4; ++g) sg[g] = __ldg(splane + c * 128 + g * 32 + lane);
    }

    // ---- A: lane bit counts
    uint32_t lane_bits = 0;
    if (fast) {
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const uint32_t w[4] = {ev[q].x, ev[q].y, ev[q].z, ev[q].w};
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int j = 4 * q + r;
          const uint32_t nib = (sg[j >> 3] >> (28 - 4 * (j & 7))) & 15u;
#pragma unroll
          for (int e = 0; e < 4; ++e) lane_bits += tb.enc[key_of(w[r], nib, e)].y;
        }
      }
    } else if (valid) {
      lane_bits = chunk_slow(tb, eplane, splane, c, lane, n, nullptr, 0);
    }
    if (valid) lane_index[c * kLanes + lane] = (uint16_t)lane_bits;
    uint32_t incl = lane_bits;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
      if ((int)lane >= d) incl += v;
    }
    const uint32_t lane_start = incl - lane_bits;
    const uint32_t chunk_bits = __shfl_sync(0xffffffffu, incl, 31);
    const uint32_t chunk_bytes = valid ? (uint32_t)align_up((chunk_bits + 7) / 8, kPayloadAlign) : 0u;
    const bool staged = chunk_bytes <= kStageWords * 4;
    if (lane == 0) s_chunk_bytes[warp] = chunk_bytes;
    __syncthreads();

    // ---- publish this tile's size as early as possible
    unsigned long long tile_bytes = 0;
#pragma unroll
    for (int w = 0; w < (int)kEncWarps; ++w) tile_bytes += s_chunk_bytes[w];
    if (tid == 0) {
      const unsigned long long flag = tile == 0 ? kTilePrefix : kTileAggregate;
      st_tile(&tiles[tile], (flag << kTileFlagShift) | tile_bytes);
      if (tile == 0) s_tile_base = 0;
    }

    // ---- B: assemble the chunk in shared memory
    if (valid && staged) {
      uint4* st4 = reinterpret_cast<uint4*>(stage);
      for (uint32_t k = lane; k < chunk_bytes / 16; k += 32) st4[k] = make_uint4(0, 0, 0, 0);
      __syncwarp();
      if (fast) {
        Packer pk{0ull, lane_start & 31u, stage + (lane_start >> 5)};
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const uint32_t w[4] = {ev[q].x, ev[q].y, ev[q].z, ev[q].w};
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const int j = 4 * q + r;
            const uint32_t nib = (sg[j >> 3] >> (28 - 4 * (j & 7))) & 15u;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint2 en = tb.enc[key_of(w[r], nib, e)];
              pk.put(en.x, en.y);
            }
          }
        }
        pk.flush();
      } else {
        chunk_slow(tb, eplane, splane, c, lane, n, stage, lane_start);
      }
    }

    // ---- C: exclusive prefix of the tile by decoupled look-back (warp 0)
    if (warp == 0 && tile > 0) {
      unsigned long long excl = 0;
      long long look = (long long)tile - 1;
      uint32_t spins = 0;
      bool abort = false;
      while (true) {
        const long long idx = look - lane;
        unsigned long long st = (kTilePrefix << kTileFlagShift);  // tiles before the first: prefix 0
        if (idx >= 0) st = ld_tile(&tiles[idx]);
        const uint32_t flag = (uint32_t)(st >> kTileFlagShift);
        const uint32_t m_prefix = __ballot_sync(0xffffffffu, flag == kTilePrefix);
        const uint32_t m_invalid = __ballot_sync(0xffffffffu, flag == kTileInvalid);
        const uint32_t m_abort = __ballot_sync(0xffffffffu, flag == kTileAbort);
        const int first_prefix = m_prefix ? __ffs(m_prefix) - 1 : 32;
        const uint32_t relevant = first_prefix < 32 ? (0xffffffffu >> (31 - first_prefix)) : 0xffffffffu;
        if (m_abort & relevant) {
          abort = true;
          break;
        }
        if (m_invalid & relevant) {
          if (++spins > kSpinLimit) {
            abort = true;
            break;
          }
          __nanosleep(40);
          continue;
        }
        unsigned long long v = ((int)lane <= first_prefix) ? (st & kTileValueMask) : 0ull;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        excl += v;
        if (first_prefix < 32) break;
        look -= 32;
      }
      if (lane == 0) {
        if (abort) {
          set_status(&ctl->status, LC_ERR_TIMEOUT);
          st_tile(&tiles[tile], kTileAbort << kTileFlagShift);
          s_abort = 1;
        } else {
          st_tile(&tiles[tile], (kTilePrefix << kTileFlagShift) | (excl + tile_bytes));
          s_tile_base = excl;
        }
      }
    }
    __syncthreads();
    if (s_abort) continue;

    // ---- D: write the chunk and its index entry
    unsigned long long chunk_off = s_tile_base;
    for (uint32_t w = 0; w < warp; ++w) chunk_off += s_chunk_bytes[w];
    if (valid) {
      if (lane == 0) chunk_index[c] = chunk_off;
      uint4* dst4 = reinterpret_cast<uint4*>(payload + chunk_off);
      if (staged) {
        __syncwarp();
        const uint4* st4 = reinterpret_cast<const uint4*>(stage);
        for (uint32_t k = lane; k < chunk_bytes / 16; k += 32) dst4[k] = st4[k];
      } else {
        // chunk larger than the staging area: OR the bits straight into (zeroed) global memory.
        for (uint32_t k = lane; k < chunk_bytes / 16; k += 32) dst4[k] = make_uint4(0, 0, 0, 0);
        __threadfence_block();
        __syncwarp();
        chunk_slow(tb, eplane, splane, c, lane, n, reinterpret_cast<uint32_t*>(dst4), lane_start);
      }
    }
    if (tile == ntiles - 1 && tid == 0) {
      const unsigned long long payload_bytes = s_tile_base + tile_bytes;
      chunk_index[nchunks] = payload_bytes;
      *reinterpret_cast<unsigned long long*>(stream + 48) = L.payload_off + payload_bytes;
    }
  }
}

}  // namespace

cudaError_t launch_encode(Control* ctl, unsigned long long* tiles, const uint8_t* eplane,
                          const uint32_t* splane, uint64_t n, uint8_t* stream, cudaStream_t cs) {
  const WorkspaceLayout W = workspace_layout(n);
  if (W.ntiles == 0) return cudaSuccess;
  static int blocks_per_sm = 0, sms = 0;
  if (blocks_per_sm == 0) {
    cudaError_t e = cudaFuncSetAttribute(encode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kEncSmem);
    if (e != cudaSuccess) return e;
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    int bps = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, encode_kernel, kEncThreads, kEncSmem);
    if (e != cudaSuccess) return e;
    blocks_per_sm = bps > 0 ? bps : 1;
  }
  const uint64_t full = (uint64_t)sms * blocks_per_sm;
  const unsigned grid = (unsigned)(W.ntiles < full ? W.ntiles : full);
  encode_kernel<<<grid, kEncThreads, kEncSmem, cs>>>(ctl, tiles, eplane, splane, n, stream);
  return cudaGetLastError();
}

}  // namespace lc
