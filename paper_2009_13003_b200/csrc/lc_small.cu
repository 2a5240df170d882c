// Small vectors: the whole compress pass (Algorithm 1 steps 4-6, optionally step 7) in one CTA and one launch.
//
// For a vector of a few chunks the three kernels of the general path and the memset before them are all launch
// latency (about 40 us together); layers of a few hundred elements are common in per-layer use. Here one CTA of 512
// threads does the statistics in shared memory, runs the table pass (the same function as table_kernel), and codes
// the chunks one warp per chunk, straight into the payload. Same bytes as the general path.
#include "lc_table.cuh"

namespace lc {
namespace {

__device__ __forceinline__ uint32_t key_of_bits(uint32_t bits) { return ((bits >> 31) << 8) | ((bits >> 23) & 255u); }

// Appends a code of at most 32 bits to a lane's bit accumulator; completed words are ORed into the zeroed payload.
struct WordPacker {
  unsigned long long acc;
  uint32_t nb;
  uint32_t* dst;
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

// Per-key tables in shared memory for the coding passes: code length, low 32 bits of the code, representative.
struct KeyTables {
  const uint32_t* len;
  const uint32_t* code;
  const EncEntry* enc;  // global: the upper code bits of the rare codes longer than 32 bits
};

// Bits of lane `lane`'s sub-stream of chunk c (format section 2); with dst != nullptr the codes are also written,
// starting at bit lane_start of the chunk image at dst. Only the steps that hold elements are visited; a lane's four
// elements of a step are read as one 16-byte vector where all four exist.
__device__ uint32_t code_lane(const KeyTables& T, const float* base, const float* cur, uint64_t n, uint64_t c,
                              uint32_t lane, uint32_t* dst, uint32_t lane_start) {
  WordPacker pk{0ull, lane_start & 31u, dst ? dst + (lane_start >> 5) : nullptr};
  uint32_t bits = 0;
  const uint64_t c0 = c * kChunkElems;
  const uint32_t in_chunk = (uint32_t)(n - c0 < kChunkElems ? n - c0 : kChunkElems);
  const uint32_t steps = (in_chunk + 127) / 128;
  for (uint32_t j = 0; j < steps; ++j) {
    const uint64_t i0 = c0 + 128ull * j + 4 * lane;
    float d[4];
    uint32_t cnt = 0;
    if (i0 + 4 <= n) {
      const float4 b4 = *reinterpret_cast<const float4*>(base + i0), c4 = *reinterpret_cast<const float4*>(cur + i0);
      d[0] = __fsub_rn(c4.x, b4.x); d[1] = __fsub_rn(c4.y, b4.y); d[2] = __fsub_rn(c4.z, b4.z); d[3] = __fsub_rn(c4.w, b4.w);
      cnt = 4;
    } else {
      for (uint32_t e = 0; e < kGroup; ++e)
        if (i0 + e < n) d[cnt++] = __fsub_rn(cur[i0 + e], base[i0 + e]);
    }
    for (uint32_t e = 0; e < cnt; ++e) {
      const uint32_t key = key_of_bits(__float_as_uint(d[e]));
      const uint32_t len = T.len[key];
      bits += len;
      if (dst) {
        if (len > 32) {
          pk.put(T.enc[key].code_hi, len - 32);
          pk.put(T.code[key], 32);
        } else {
          pk.put(T.code[key], len);
        }
      }
    }
  }
  if (dst) pk.flush();
  return bits;
}

constexpr uint32_t kSmallWarps = kTableThreads / 32;  // one chunk per warp
static_assert(kSmallMaxElems <= (uint64_t)kSmallWarps * kChunkElems, "a warp per chunk");

__global__ void __launch_bounds__(kTableThreads)
small_compress_kernel(Control* ctl, const float* base, const float* cur, uint64_t n, int nbits, uint8_t* stream,
                      float* tracked_out, int keep_status) {
  __shared__ uint32_t h_count[kKeys], h_inv_min[kKeys], h_max[kKeys];
  __shared__ uint32_t s_chunk_bytes[kSmallWarps];
  __shared__ unsigned long long s_chunk_off[kSmallWarps + 1];
  __shared__ uint32_t s_lane_start[kSmallWarps][32];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- what the memset of the general path clears, as far as this kernel uses it
  if (tid == 0) {
    if (!keep_status) ctl->status = 0;
    ctl->ticket = 0;
    ctl->nsym = 0;
    ctl->max_len = 0;
    ctl->payload_bits = 0;
    ctl->wide = 0;
  }
  h_count[tid] = 0;
  h_inv_min[tid] = 0;
  h_max[tid] = 0;
  __syncthreads();

  // ---- statistics (Section 3.1.1): count, and the running maxima of ~bits and bits, per key
  // (Finding the lanes of a warp that meet the same key with a match, so that one lane updates the bin for all of
  // them, was measured slower than these plain shared-memory atomics: 57 against 45 us at 4096 elements.)
  for (uint64_t i = tid; i < n; i += kTableThreads) {
    const uint32_t bits = __float_as_uint(__fsub_rn(cur[i], base[i]));
    const uint32_t key = key_of_bits(bits);
    atomicAdd(&h_count[key], 1u);
    atomicMax(&h_inv_min[key], ~bits);
    atomicMax(&h_max[key], bits);
  }
  __syncthreads();
  ctl->count[tid] = h_count[tid];
  ctl->inv_min[tid] = h_inv_min[tid];
  ctl->max_bits[tid] = h_max[tid];
  ctl->mant_sum[tid] = 0;
  __syncthreads();  // this CTA's own global writes are visible to all its threads

  // ---- table pass: header, symbol table, per-key encode table
  if (!table_pass(ctl, n, nbits, stream, /*wide_ok=*/1, /*fixed=*/0, nullptr, nullptr, /*mean=*/0)) return;
  __syncthreads();

  // ---- encode: lane bit counts and chunk sizes, then the chunk offsets, then the bits
  // the statistics are in the control block now: their shared arrays take the per-key tables of the coding passes
  const EncEntry* enc = ctl->enc;
  uint32_t *k_len = h_count, *k_code = h_inv_min, *k_rep = h_max;
  {
    const EncEntry e = enc[tid];
    k_len[tid] = e.len;
    k_code[tid] = e.code_lo;
    k_rep[tid] = *reinterpret_cast<const uint32_t*>(stream + kHeaderBytes + kTableEntryBytes * e.sym + 4);
  }
  __syncthreads();
  const KeyTables T{k_len, k_code, enc};
  const StreamLayout L = stream_layout(n, ctl->nsym);
  const uint32_t nchunks = (uint32_t)L.nchunks;  // at most kSmallWarps (checked by the launcher)
  unsigned long long* chunk_index = reinterpret_cast<unsigned long long*>(stream + L.chunk_index_off);
  uint16_t* lane_index = reinterpret_cast<uint16_t*>(stream + L.lane_index_off);
  uint8_t* payload = stream + L.payload_off;
  if (warp < nchunks) {
    const uint32_t bits = code_lane(T, base, cur, n, warp, lane, nullptr, 0);
    lane_index[warp * kLanes + lane] = (uint16_t)bits;
    uint32_t incl = bits;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
      if ((int)lane >= d) incl += v;
    }
    s_lane_start[warp][lane] = incl - bits;
    if (lane == 31) s_chunk_bytes[warp] = (uint32_t)align_up((incl + 7) / 8, kPayloadAlign);
  }
  __syncthreads();
  if (tid == 0) {
    unsigned long long off = 0;
    for (uint32_t c = 0; c < nchunks; ++c) {
      s_chunk_off[c] = off;
      chunk_index[c] = off;
      off += s_chunk_bytes[c];
    }
    s_chunk_off[nchunks] = off;
    chunk_index[nchunks] = off;
    *reinterpret_cast<unsigned long long*>(stream + 48) = L.payload_off + off;
  }
  __syncthreads();
  if (warp < nchunks) {
    uint4* dst4 = reinterpret_cast<uint4*>(payload + s_chunk_off[warp]);
    for (uint32_t k = lane; k < s_chunk_bytes[warp] / 16; k += 32) dst4[k] = make_uint4(0, 0, 0, 0);
    __syncwarp();  // the zeros are in place before any lane ORs into them
    code_lane(T, base, cur, n, warp, lane, reinterpret_cast<uint32_t*>(dst4), s_lane_start[warp][lane]);
  }

  // ---- Algorithm 1 step 7: tracked_out = base + quantized delta (tracked_out may be base: everything that reads
  // base for coding is done)
  if (tracked_out) {
    __syncthreads();
    for (uint64_t i = tid; i < n; i += kTableThreads) {
      const float b = base[i];
      tracked_out[i] = __fadd_rn(b, __uint_as_float(k_rep[key_of_bits(__float_as_uint(__fsub_rn(cur[i], b)))]));
    }
  }
}

}  // namespace

cudaError_t launch_small_compress(Control* ctl, const float* base, const float* cur, uint64_t n, int nbits,
                                  uint8_t* stream, float* tracked_out, bool keep_status, cudaStream_t cs) {
  if (n == 0 || n > kSmallMaxElems) return cudaErrorInvalidValue;
  small_compress_kernel<<<1, kTableThreads, 0, cs>>>(ctl, base, cur, n, nbits, stream, tracked_out, keep_status ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace lc
