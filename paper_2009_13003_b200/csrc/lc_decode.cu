// Recovery pass: chunk-parallel Huffman decode of up to four streams fused with the chain add.
//
// Paper: the reconstruction identity u_t = u_0 + sum of the quantized deltas (Section 3, after
// component C2) and Algorithm 1 step 7 (tracked state += quantized delta), applied k times left to
// right in fp32. Stream layout: format text sections 2-4.
//
// One warp decodes one chunk; lane t walks lane sub-stream t of every stream at once, so at step j
// the warp holds 128 consecutive elements: one coalesced 16-byte load of base and one 16-byte store of
// out per lane, with the k representatives added in registers in between. Codes are looked up in a
// shared-memory table indexed by the next kLutBits bits whose entries hold the representative value
// itself; longer codes take a canonical first-code search.
//
// Every read of a stream is bounds-checked against the caller's buffer size and every table is
// validated before use, so a damaged stream yields LC_ERR_FORMAT (and unspecified output), never an
// out-of-bounds access.
//
// Bound: HBM at k = 1 (8 bytes per element + the stream); at k = 4 the integer work per symbol is
// the limit.
#include "lc_common.cuh"

namespace lc {
namespace {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kLutBits = 10;
constexpr uint32_t kLongCode = 0xFFFFFFFFu;

struct StreamState {
  uint2 lut[1 << kLutBits];          // {bit pattern of rep, code length}; length kLongCode = longer code
  uint32_t sorted_rep[256];          // representatives in canonical (len, id) order
  unsigned long long first_code[64]; // first canonical code of each length
  uint32_t len_count[64];            // codes of each length
  uint32_t len_offset[64];           // index of the first of them in sorted_rep
  // header
  unsigned long long n, payload_bits, total_bytes, payload_off, payload_size;
  unsigned long long chunk_index_off, lane_index_off;
  uint32_t nsym, max_len, nchunks, only_rep;
  // validation accumulators
  unsigned long long kraft, count_sum, bit_sum;
  uint32_t seen_max, nused;
};

__device__ __forceinline__ uint64_t load_le(const uint8_t* p, int bytes) {
  uint64_t v = 0;
  for (int b = 0; b < bytes; ++b) v |= (uint64_t)p[b] << (8 * b);
  return v;
}

// Parses and validates stream `s`, then builds its decode tables in shared memory. All threads of the
// CTA call this; returns 0 or the error to report.
__device__ int prepare_stream(StreamState& S, const uint8_t* __restrict__ s, uint64_t bytes, uint64_t n,
                              int* s_err) {
  const int tid = threadIdx.x;
  if (tid == 0) {
    int err = 0;
    S.kraft = 0; S.count_sum = 0; S.bit_sum = 0; S.seen_max = 0; S.nused = 0; S.only_rep = 0;
    if (bytes < kHeaderBytes) {
      err = LC_ERR_FORMAT;
    } else {
      const uint32_t nbits = s[6];
      S.n = load_le(s + 8, 8);
      S.nsym = (uint32_t)load_le(s + 16, 4);
      S.max_len = (uint32_t)load_le(s + 20, 4);
      S.nchunks = (uint32_t)load_le(s + 32, 4);
      S.payload_bits = load_le(s + 40, 8);
      S.total_bytes = load_le(s + 48, 8);
      S.payload_off = load_le(s + 56, 8);
      const bool magic = s[0] == 'L' && s[1] == 'C' && s[2] == 'C' && s[3] == '1';
      if (!magic || load_le(s + 4, 2) != 1 || nbits < 1 || nbits > 8 || s[7] != 0) err = LC_ERR_FORMAT;
      else if (S.nsym < 1 || S.nsym > (1u << nbits) || S.max_len > 63) err = LC_ERR_FORMAT;
      else if (load_le(s + 24, 4) != kChunkElems || load_le(s + 28, 2) != kLanes ||
               load_le(s + 30, 2) != kGroup || load_le(s + 36, 4) != kPayloadAlign) err = LC_ERR_FORMAT;
      else if (S.n != n) err = S.n < (1ull << 32) ? LC_ERR_MISMATCH : LC_ERR_FORMAT;
      if (!err) {
        const StreamLayout L = stream_layout(S.n, S.nsym);
        S.chunk_index_off = L.chunk_index_off;
        S.lane_index_off = L.lane_index_off;
        if (S.nchunks != L.nchunks || S.payload_off != L.payload_off || S.total_bytes > bytes ||
            S.total_bytes < L.payload_off) {
          err = LC_ERR_FORMAT;
        } else {
          S.payload_size = S.total_bytes - S.payload_off;
          if (load_le(s + L.chunk_index_off, 8) != 0 ||
              load_le(s + L.chunk_index_off + 8 * L.nchunks, 8) != S.payload_size)
            err = LC_ERR_FORMAT;
        }
      }
    }
    *s_err = err;
  }
  for (int L = tid; L < 64; L += kDecThreads) S.len_count[L] = 0;
  __syncthreads();
  if (*s_err) return *s_err;

  // ---- table entries: one thread per symbol
  const uint32_t nsym = S.nsym;
  uint32_t my_len = 0, my_rep = 0;
  unsigned long long my_count = 0;
  bool entry_bad = false;
  if (tid < (int)nsym) {
    const uint8_t* e = s + kHeaderBytes + kTableEntryBytes * tid;
    my_len = e[2];
    my_rep = (uint32_t)load_le(e + 4, 4);
    my_count = load_le(e + 8, 8);
    entry_bad = e[3] != 0 || my_len > 63 || (my_count == 0 && my_len != 0);
    if (my_count != 0) {
      atomicAdd(&S.count_sum, my_count);
      atomicAdd(&S.bit_sum, my_count * my_len);
      atomicAdd(&S.nused, 1u);
      atomicMax(&S.seen_max, my_len);
      S.only_rep = my_rep;  // meaningful only when a single symbol is used
      if (my_len > 0 && my_len <= 63) {
        atomicAdd(&S.kraft, 1ull << (63 - my_len));
        atomicAdd(&S.len_count[my_len], 1u);
      }
    }
  }
  if (__syncthreads_or(entry_bad)) return LC_ERR_FORMAT;
  if (tid == 0) {
    int err = 0;
    if (S.count_sum != S.n || S.bit_sum != S.payload_bits || S.seen_max != S.max_len) err = LC_ERR_FORMAT;
    if (S.nused >= 2) {
      if (S.kraft != (1ull << 63)) err = LC_ERR_FORMAT;
    } else if (S.max_len != 0) {
      err = LC_ERR_FORMAT;
    }
    // canonical first codes per length
    unsigned long long code = 0;
    uint32_t offset = 0;
    for (int L = 1; L < 64; ++L) {
      S.first_code[L] = code;
      S.len_offset[L] = offset;
      code = (code + S.len_count[L]) << 1;
      offset += S.len_count[L];
    }
    S.first_code[0] = 0;
    S.len_offset[0] = 0;
    *s_err = err;
  }
  __syncthreads();
  if (*s_err) return *s_err;
  if (S.nused >= 2 && tid < (int)nsym && my_count != 0) {
    // rank among the symbols of the same length with smaller id (zero-count symbols have length 0)
    uint32_t r = 0;
    for (int j = 0; j < tid; ++j) r += (s[kHeaderBytes + kTableEntryBytes * j + 2] == my_len) ? 1u : 0u;
    S.sorted_rep[S.len_offset[my_len] + r] = my_rep;
  }
  __syncthreads();

  // ---- lookup table: one thread per entry, canonical decode of the entry's own index
  for (uint32_t idx = tid; idx < (1u << kLutBits); idx += kDecThreads) {
    uint2 ent = make_uint2(0u, kLongCode);
    if (S.nused < 2) {
      ent = make_uint2(S.only_rep, 0u);
    } else {
      for (uint32_t L = 1; L <= (uint32_t)kLutBits; ++L) {
        const unsigned long long c = idx >> (kLutBits - L);
        if (c >= S.first_code[L] && c - S.first_code[L] < S.len_count[L]) {
          ent = make_uint2(S.sorted_rep[S.len_offset[L] + (uint32_t)(c - S.first_code[L])], L);
          break;
        }
      }
    }
    S.lut[idx] = ent;
  }
  __syncthreads();
  return 0;
}

// Bounded word read of a chunk's payload.
struct ChunkReader {
  const uint32_t* words;
  uint32_t nwords;
  __device__ __forceinline__ uint32_t rd(uint32_t i) const { return i < nwords ? __ldg(words + i) : 0u; }
};

// Canonical search for a code longer than kLutBits, from bit position p of word wi.
__device__ __noinline__ uint2 decode_long(const StreamState& S, const uint32_t* words, uint32_t nwords,
                                          uint32_t wi, uint32_t p, int32_t* status) {
  const ChunkReader R{words, nwords};
  const unsigned long long a = ((unsigned long long)R.rd(wi) << 32) | R.rd(wi + 1);
  const unsigned long long b = R.rd(wi + 2);
  const unsigned long long window = p ? ((a << p) | (b >> (32 - p))) : a;
  for (uint32_t L = kLutBits + 1; L <= S.max_len; ++L) {
    const unsigned long long c = window >> (64 - L);
    if (c >= S.first_code[L] && c - S.first_code[L] < S.len_count[L])
      return make_uint2(S.sorted_rep[S.len_offset[L] + (uint32_t)(c - S.first_code[L])], L);
  }
  set_status(status, LC_ERR_FORMAT);  // no code matches: damaged payload
  return make_uint2(0u, S.max_len ? S.max_len : 1u);
}

struct LaneCursor {
  ChunkReader R;
  uint32_t wi;      // index of w0
  uint32_t p;       // bit position inside w0
  uint32_t w0, w1;  // current and next word
};

template <int KS>
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(const float* base, DecodeStreams streams, uint64_t n, float* out,
              int32_t* __restrict__ status) {
  __shared__ StreamState S[KS];
  __shared__ int s_err;

#pragma unroll
  for (int s = 0; s < KS; ++s) {
    const int err = prepare_stream(S[s], streams.ptr[s], streams.bytes[s], n, &s_err);
    if (err) {
      if (threadIdx.x == 0) set_status(status, err);
      return;
    }
  }

  const uint32_t lane = threadIdx.x & 31;
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  const uint64_t warp0 = (uint64_t)blockIdx.x * kDecWarps + (threadIdx.x >> 5);
  const uint64_t nwarps = (uint64_t)gridDim.x * kDecWarps;

  for (uint64_t c = warp0; c < nchunks; c += nwarps) {
    LaneCursor cur[KS];
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint8_t* sp = streams.ptr[s];
      const unsigned long long* ci = reinterpret_cast<const unsigned long long*>(sp + S[s].chunk_index_off);
      unsigned long long off0 = __ldg(ci + c), off1 = __ldg(ci + c + 1);
      if (off0 > off1 || off1 > S[s].payload_size || (off0 & 3) || (off1 & 3)) {
        set_status(status, LC_ERR_FORMAT);
        off0 = off1 = 0;
      }
      cur[s].R.words = reinterpret_cast<const uint32_t*>(sp + S[s].payload_off + off0);
      cur[s].R.nwords = (uint32_t)((off1 - off0) >> 2);
      const uint16_t* li = reinterpret_cast<const uint16_t*>(sp + S[s].lane_index_off);
      const uint32_t lane_bits = __ldg(li + c * kLanes + lane);
      uint32_t incl = lane_bits;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
        if ((int)lane >= d) incl += v;
      }
      const uint32_t start = incl - lane_bits;
      cur[s].wi = start >> 5;
      cur[s].p = start & 31;
      cur[s].w0 = cur[s].R.rd(cur[s].wi);
      cur[s].w1 = cur[s].R.rd(cur[s].wi + 1);
    }

    const uint64_t e0 = c * kChunkElems + 4 * lane;
    const bool full = (c + 1) * kChunkElems <= n;
    for (uint32_t j = 0; j < kSteps; ++j) {
      const uint64_t i = e0 + 128ull * j;
      float x[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t nvalid = 4;
      if (full) {
        const float4 b = __ldcs(reinterpret_cast<const float4*>(base + i));
        x[0] = b.x; x[1] = b.y; x[2] = b.z; x[3] = b.w;
      } else {
        nvalid = i >= n ? 0u : (uint32_t)min((unsigned long long)4, (unsigned long long)(n - i));
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((uint32_t)e < nvalid) x[e] = base[i + e];
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (!full && (uint32_t)e >= nvalid) break;
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          LaneCursor& C = cur[s];
          const uint32_t peek = __funnelshift_l(C.w1, C.w0, C.p);
          uint2 ent = S[s].lut[peek >> (32 - kLutBits)];
          if (ent.y == kLongCode) ent = decode_long(S[s], C.R.words, C.R.nwords, C.wi, C.p, status);
          x[e] = __fadd_rn(x[e], __uint_as_float(ent.x));
          C.p += ent.y;
          while (C.p >= 32) {
            C.p -= 32;
            C.wi += 1;
            C.w0 = C.w1;
            C.w1 = C.R.rd(C.wi + 1);
          }
        }
      }
      if (full) {
        __stcs(reinterpret_cast<float4*>(out + i), make_float4(x[0], x[1], x[2], x[3]));
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((uint32_t)e < nvalid) out[i + e] = x[e];
      }
    }
  }
}

template <int KS>
cudaError_t launch_decode_ks(const float* base, const DecodeStreams& streams, uint64_t n, float* out,
                             int32_t* status, cudaStream_t cs) {
  static int blocks_per_sm = 0, sms = 0;
  if (blocks_per_sm == 0) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    int bps = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, decode_kernel<KS>, kDecThreads, 0);
    if (e != cudaSuccess) return e;
    blocks_per_sm = bps > 0 ? bps : 1;
  }
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  uint64_t want = (nchunks + kDecWarps - 1) / kDecWarps;
  if (want == 0) want = 1;  // still validates the streams
  const uint64_t full = (uint64_t)sms * blocks_per_sm;
  const unsigned grid = (unsigned)(want < full ? want : full);
  decode_kernel<KS><<<grid, kDecThreads, 0, cs>>>(base, streams, n, out, status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode(const float* base, const DecodeStreams& streams, int k, uint64_t n, float* out,
                          int32_t* status, cudaStream_t cs) {
  switch (k) {
    case 1: return launch_decode_ks<1>(base, streams, n, out, status, cs);
    case 2: return launch_decode_ks<2>(base, streams, n, out, status, cs);
    case 3: return launch_decode_ks<3>(base, streams, n, out, status, cs);
    case 4: return launch_decode_ks<4>(base, streams, n, out, status, cs);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace lc
