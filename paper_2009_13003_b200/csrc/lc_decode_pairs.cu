// Recovery pass for streams of at most 32 symbols (priority promotion with x <= 5 bits, the range the paper
// evaluates): chunk-parallel Huffman decode that resolves TWO symbols per table lookup, fused with the chain add.
//
// Paper: the reconstruction identity u_t = u_0 + sum of the quantized deltas (Section 3, after component C2) and
// Algorithm 1 step 7, applied k times left to right in fp32. Stream layout: format text sections 2-4.
//
// Work split as in the general decoder (lc_decode.cu): one warp per chunk, lane t walks lane sub-stream t of all
// k streams at once, one coalesced 16-byte load of base and store of out per lane and step. What differs is the
// inner loop, which is bound by instruction issue and by the shared-memory pipe, not by HBM, at k = 4:
//
//  * One table per stream, indexed by the next 13 bits, 16-bit entries: the symbols of the next TWO codes and
//    the bits both take, when both fit the 13 bits (99.5 % of the pairs on the log-normal workload). A lookup,
//    a shift of the bit buffer and one top-up test then serve two elements instead of one.
//  * The representative is not in the table (two of them do not fit an entry that small): lane j of the warp
//    keeps representative j of every stream in a register, and a symbol's value is fetched with a warp shuffle.
//    That is what limits this path to 32 symbols.
//  * A pair that does not fit (or a first code longer than 13 bits) carries a mark; one warp vote per pair sends
//    the warp through a short handler in which the marked lanes decode their two codes one by one (table again
//    for codes up to 13 bits, canonical search beyond).
//  * A lane tops its 64-bit bit buffer up once per step (4 elements): two pair lookups take at most 26 bits.
//
// The tables are built once per call by decode_prepare_kernel (one CTA per stream, which also validates the
// stream: header, symbol table, Kraft sum, counts) and left in the workspace; every CTA of the decode kernel
// copies them into its shared memory. The prepare kernel also decides which decode kernel runs: a flag word in
// the workspace tells this kernel, or the general one, to return at once.
//
// Every read of a stream is bounds-checked against the caller's buffer size, so a damaged stream yields
// LC_ERR_FORMAT (and unspecified output), never an out-of-bounds access.
#include "lc_decode_bits.cuh"

namespace lc {
namespace {

using namespace dec;

constexpr int kPrepThreads = 256;
constexpr int kDecMaxThreads = 512;
constexpr int kPairBits = 13;
constexpr uint32_t kPairEntries = 1u << kPairBits;
// 16-bit entry: symbol A in bits 0-4, symbol B in bits 5-9, kPairLong, kPairExc, bits consumed in bits 12-15.
constexpr uint32_t kPairLong = 0x0400;  // the first code is longer than 13 bits (always with kPairExc)
constexpr uint32_t kPairExc = 0x0800;   // the entry does not resolve two symbols; bits 12-15 = length of the first
constexpr uint32_t kMaxPairSyms = 32;

struct PairAux {
  uint32_t rep[kMaxPairSyms];            // representative (bit pattern) by symbol id
  uint8_t len[kMaxPairSyms];             // code length by symbol id
  uint8_t sorted_sym[kMaxPairSyms];      // symbol ids in canonical (len, id) order
  unsigned long long first_code[64];     // first canonical code of each length
  unsigned long long last_aligned[64];   // largest left-aligned 64-bit window whose code has at most this length
  uint32_t len_count[64];                // codes of each length
  uint32_t len_offset[64];               // index of the first of them in sorted_sym
  unsigned long long payload_off, payload_size, chunk_index_off, lane_index_off;
  uint32_t nsym, max_len, nused, only_sym;
};
struct alignas(16) PairStream {
  uint16_t pair[kPairEntries];
  PairAux aux;
};
static_assert(sizeof(PairStream) % 16 == 0, "copied with 16-byte accesses");
static_assert(sizeof(PairStream) * 4 <= kDecodeTableBytes, "the workspace region holds the tables of four streams");

// Canonical decode of the top `width` bits `idx`: (index into sorted_sym, length) or length 0 if no code of at
// most `width` bits matches.
__device__ __forceinline__ uint2 canonical_lookup(const PairAux& A, uint32_t idx, uint32_t width) {
  for (uint32_t L = 1; L <= width; ++L) {
    const unsigned long long c = idx >> (width - L);
    if (c >= A.first_code[L] && c - A.first_code[L] < A.len_count[L])
      return make_uint2(A.len_offset[L] + (uint32_t)(c - A.first_code[L]), L);
  }
  return make_uint2(0u, 0u);
}

// One CTA per stream: validates the stream (format section 4) and, if it has at most 32 symbols, builds its pair
// table. Sets kDecodeFlagError / kDecodeFlagGeneral in *flags and the status word on error.
__global__ void __launch_bounds__(kPrepThreads)
decode_prepare_kernel(DecodeStreams streams, uint64_t n, PairStream* __restrict__ tables, uint32_t* __restrict__ flags,
                      int32_t* __restrict__ status) {
  __shared__ PairAux A;
  __shared__ alignas(16) uint8_t hdr[kHeaderBytes];
  __shared__ unsigned long long s_kraft, s_count_sum, s_bit_sum, s_n, s_payload_bits;
  __shared__ uint32_t s_seen_max;
  __shared__ int s_err;

  const int tid = threadIdx.x;
  const uint8_t* __restrict__ s = streams.ptr[blockIdx.x];
  const uint64_t bytes = streams.bytes[blockIdx.x];
  if (tid < 4 && bytes >= kHeaderBytes) reinterpret_cast<uint4*>(hdr)[tid] = __ldg(reinterpret_cast<const uint4*>(s) + tid);
  for (int L = tid; L < 64; L += kPrepThreads) A.len_count[L] = 0;
  if (tid < (int)kMaxPairSyms) {
    A.rep[tid] = 0;
    A.len[tid] = 0;
    A.sorted_sym[tid] = 0;
  }
  __syncthreads();
  if (tid == 0) {
    int err = 0;
    const uint8_t* h = hdr;
    s_kraft = 0; s_count_sum = 0; s_bit_sum = 0; s_seen_max = 0;
    A.nused = 0; A.only_sym = 0; A.nsym = 0; A.max_len = 0;
    if (bytes < kHeaderBytes) {
      err = LC_ERR_FORMAT;
    } else {
      const uint32_t nbits = h[6];
      s_n = load_le(h + 8, 8);
      A.nsym = (uint32_t)load_le(h + 16, 4);
      A.max_len = (uint32_t)load_le(h + 20, 4);
      const uint32_t nchunks = (uint32_t)load_le(h + 32, 4);
      s_payload_bits = load_le(h + 40, 8);
      const unsigned long long total_bytes = load_le(h + 48, 8);
      A.payload_off = load_le(h + 56, 8);
      const bool magic = h[0] == 'L' && h[1] == 'C' && h[2] == 'C' && h[3] == '1';
      if (!magic || load_le(h + 4, 2) != 1 || nbits < 1 || nbits > 8 || h[7] != 0) err = LC_ERR_FORMAT;
      else if (A.nsym < 1 || A.nsym > (1u << nbits) || A.max_len > 63) err = LC_ERR_FORMAT;
      else if (load_le(h + 24, 4) != kChunkElems || load_le(h + 28, 2) != kLanes ||
               load_le(h + 30, 2) != kGroup || load_le(h + 36, 4) != kPayloadAlign) err = LC_ERR_FORMAT;
      else if (s_n != n) err = s_n < (1ull << 32) ? LC_ERR_MISMATCH : LC_ERR_FORMAT;
      if (!err) {
        const StreamLayout L = stream_layout(s_n, A.nsym);
        A.chunk_index_off = L.chunk_index_off;
        A.lane_index_off = L.lane_index_off;
        if (nchunks != L.nchunks || A.payload_off != L.payload_off || total_bytes > bytes ||
            total_bytes < L.payload_off) {
          err = LC_ERR_FORMAT;
        } else {
          A.payload_size = total_bytes - A.payload_off;
          if (load_le(s + L.chunk_index_off, 8) != 0 ||
              load_le(s + L.chunk_index_off + 8 * L.nchunks, 8) != A.payload_size)
            err = LC_ERR_FORMAT;
        }
      }
    }
    s_err = err;
  }
  __syncthreads();
  if (s_err) {
    if (tid == 0) {
      set_status(status, s_err);
      atomicOr(flags, kDecodeFlagError);
    }
    return;
  }
  if (A.nsym > kMaxPairSyms) {
    // the general decode kernel validates the symbol table itself
    if (tid == 0) atomicOr(flags, kDecodeFlagGeneral);
    return;
  }

  // ---- symbol table: one thread per symbol
  const uint32_t nsym = A.nsym;
  uint32_t my_len = 0;
  unsigned long long my_count = 0;
  bool entry_bad = false;
  if (tid < (int)nsym) {
    const uint4 e = __ldg(reinterpret_cast<const uint4*>(s + kHeaderBytes) + tid);  // key:16 len:8 pad:8 | rep | count
    my_len = (e.x >> 16) & 255u;
    my_count = ((unsigned long long)e.w << 32) | e.z;
    entry_bad = (e.x >> 24) != 0 || my_len > 63 || (my_count == 0 && my_len != 0);
    A.rep[tid] = e.y;
    A.len[tid] = (uint8_t)my_len;
    if (my_count != 0) {
      atomicAdd(&s_count_sum, my_count);
      atomicAdd(&s_bit_sum, my_count * my_len);
      atomicAdd(&A.nused, 1u);
      atomicMax(&s_seen_max, my_len);
      A.only_sym = tid;  // meaningful only when a single symbol is used
      if (my_len > 0 && my_len <= 63) {
        atomicAdd(&s_kraft, 1ull << (63 - my_len));
        atomicAdd(&A.len_count[my_len], 1u);
      }
    }
  }
  const int any_bad = __syncthreads_or(entry_bad);
  if (tid == 0) {
    int err = any_bad ? LC_ERR_FORMAT : 0;
    if (s_count_sum != s_n || s_bit_sum != s_payload_bits || s_seen_max != A.max_len) err = LC_ERR_FORMAT;
    if (A.nused >= 2) {
      if (s_kraft != (1ull << 63)) err = LC_ERR_FORMAT;
    } else if (A.max_len != 0) {
      err = LC_ERR_FORMAT;
    }
    // canonical first codes per length; codes of length <= L fill the left-aligned range
    // [0, (first_code[L] + count[L]) << (64 - L))
    unsigned long long code = 0;
    uint32_t offset = 0;
    A.first_code[0] = 0;
    A.len_offset[0] = 0;
    A.last_aligned[0] = 0;
    for (int L = 1; L < 64; ++L) {
      A.first_code[L] = code;
      A.len_offset[L] = offset;
      const unsigned long long end = (code + A.len_count[L]) << (64 - L);  // 0 when the range is everything
      A.last_aligned[L] = end - 1;
      code = (code + A.len_count[L]) << 1;
      offset += A.len_count[L];
    }
    s_err = err;
  }
  __syncthreads();
  if (s_err) {
    if (tid == 0) {
      set_status(status, s_err);
      atomicOr(flags, kDecodeFlagError);
    }
    return;
  }
  if (A.nused >= 2 && tid < (int)nsym && my_count != 0) {
    // rank among the symbols of the same length with smaller id (zero-count symbols have length 0)
    uint32_t r = 0;
    for (int j = 0; j < tid; ++j) r += (A.len[j] == my_len) ? 1u : 0u;
    A.sorted_sym[A.len_offset[my_len] + r] = (uint8_t)tid;
  }
  __syncthreads();

  // ---- pair table: the entry of index i decodes the 13 bits i
  PairStream& T = tables[blockIdx.x];
  for (uint32_t i = tid; i < kPairEntries; i += kPrepThreads) {
    uint32_t ent;
    if (A.nused < 2) {
      ent = A.only_sym | (A.only_sym << 5);  // no code has a length: nothing is consumed
    } else {
      const uint2 a = canonical_lookup(A, i, kPairBits);
      if (a.y == 0) {
        ent = kPairExc | kPairLong;
      } else {
        const uint32_t rem = kPairBits - a.y;
        const uint2 b = rem ? canonical_lookup(A, i & ((1u << rem) - 1u), rem) : make_uint2(0u, 0u);
        const uint32_t sym_a = A.sorted_sym[a.x];
        if (b.y == 0) ent = sym_a | kPairExc | (a.y << 12);
        else ent = sym_a | ((uint32_t)A.sorted_sym[b.x] << 5) | ((a.y + b.y) << 12);
      }
    }
    T.pair[i] = (uint16_t)ent;
  }
  for (uint32_t i = tid; i < sizeof(PairAux) / 4; i += kPrepThreads)
    reinterpret_cast<uint32_t*>(&T.aux)[i] = reinterpret_cast<const uint32_t*>(&A)[i];
}

// ---- the decode kernel --------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

// Pair-table entry of the 13 bits at the top of `hi`. `tbl` = shared address of the first stream's table; the
// other streams' tables follow at multiples of sizeof(PairStream), which reach the load as an immediate offset.
// The index scaling is a multiply-add so that it runs beside the shifts instead of competing with them.
template <int OFFSET>
__device__ __forceinline__ uint32_t lookup_pair(uint32_t hi, uint32_t tbl) {
  uint32_t e;
  asm volatile("{\n\t"
      ".reg .u32 t, a;\n\t"
      "shr.u32 t, %1, %3;\n\t"
      "mad.lo.u32 a, t, 2, %2;\n\t"
      "ld.shared.u16 %0, [a+%4];\n\t"
      "}"
      : "=r"(e)
      : "r"(hi), "r"(tbl), "n"(32 - kPairBits), "n"(OFFSET));
  return e;
}

// Code longer than the table's 13 bits: canonical search on a 64-bit window read from the staged chunk, then
// re-seat the lane's bit buffer behind the code. Returns the symbol.
__device__ __forceinline__ uint32_t long_symbol(LaneBits<true>& B, const PairAux& A, const Source& W, int32_t* status) {
  const uint32_t pos = B.bitpos(W);
  const uint32_t idx = pos >> 5, sh = pos & 31;
  const uint32_t w0 = B.word(W, idx), w1 = B.word(W, idx + 1), w2 = B.word(W, idx + 2);
  const unsigned long long window =
      ((unsigned long long)__funnelshift_l(w1, w0, sh) << 32) | __funnelshift_l(w2, w1, sh);
  uint32_t L = kPairBits + 1;
  while (L < A.max_len && (A.len_count[L] == 0 || window > A.last_aligned[L])) L += 1;
  const unsigned long long code = window >> (64 - L);
  uint32_t sym = 0;
  if (L <= A.max_len && code >= A.first_code[L] && code - A.first_code[L] < A.len_count[L]) {
    sym = A.sorted_sym[A.len_offset[L] + (uint32_t)(code - A.first_code[L])];
  } else {
    set_status(status, LC_ERR_FORMAT);  // no code matches: damaged payload
  }
  B.seek(W, pos + L);
  return sym;
}

// The marked lanes of a pair: both codes one at a time. On return sa, sb hold the two symbols and the buffer is
// behind them, topped up so that the rest of the step finds its bits.
__device__ __forceinline__ void slow_pair(LaneBits<true>& B, const PairStream& S, uint32_t tbl, const Source& W,
                                          uint32_t e, uint32_t& sa, uint32_t& sb, int32_t* status) {
  if (e & kPairLong) {
    sa = long_symbol(B, S.aux, W, status);
  } else {
    sa = e & 31u;
    B.consume(e >> 12);  // a marked entry carries the length of its first code
  }
  B.refill(W);
  const uint32_t e2 = lds_u16(tbl + (B.hi >> (32 - kPairBits)) * 2u);
  if (e2 & kPairLong) {
    sb = long_symbol(B, S.aux, W, status);
  } else {
    sb = e2 & 31u;
    B.consume(S.aux.len[sb]);
  }
}

// Full chunk, all payloads staged: the hot loop. Per step a lane decodes 4 elements x KS streams, two elements
// per lookup; the KS streams are independent dependency chains and are written interleaved.
// Bit budget of a lane and stream: the top-up at the start of a step leaves at least 33 valid bits; a lookup
// needs 13 and takes at most 13, so the second lookup still finds 20 and the step ends with at least 7, from
// which one more word makes 39. The handler for marked pairs tops up itself.
template <int KS>
__device__ __forceinline__ void decode_chunk_pairs(const PairStream* S, const Source* W, const uint32_t* start,
                                                   const uint32_t* rep, const float* base, float* out, uint64_t c,
                                                   uint32_t lane, int32_t* status) {
  LaneBits<true> bits[KS];
  const uint32_t tbl = smem_addr(S[0].pair);
#pragma unroll
  for (int s = 0; s < KS; ++s) bits[s].seek(W[s], start[s]);
  const uint64_t e0 = c * kChunkElems + 4 * lane;
  float4 b = ldg_stream_v4(base + e0);
#pragma unroll 1
  for (uint32_t j = 0; j < kSteps; ++j) {
    const uint64_t i = e0 + 128ull * j;
    float x[4] = {b.x, b.y, b.z, b.w};
    // next step's 16 bytes of base, requested a whole step ahead (the last step re-reads its own)
    b = ldg_stream_v4(base + i + (j + 1 < kSteps ? 128 : 0));
#pragma unroll
    for (int s = 0; s < KS; ++s) bits[s].refill(W[s]);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t e[KS];
      e[0] = lookup_pair<0>(bits[0].hi, tbl);
      if (KS > 1) e[1 % KS] = lookup_pair<1 * (int)sizeof(PairStream)>(bits[1 % KS].hi, tbl);
      if (KS > 2) e[2 % KS] = lookup_pair<2 * (int)sizeof(PairStream)>(bits[2 % KS].hi, tbl);
      if (KS > 3) e[3 % KS] = lookup_pair<3 * (int)sizeof(PairStream)>(bits[3 % KS].hi, tbl);
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        uint32_t sa = e[s], sb = e[s] >> 5, used = e[s] >> 12;  // the shuffles below read the low five bits only
        if (__builtin_expect(__any_sync(0xffffffffu, (e[s] & kPairExc) != 0u), 0)) {
          if (e[s] & kPairExc) {
            slow_pair(bits[s], S[s], tbl + s * (uint32_t)sizeof(PairStream), W[s], e[s], sa, sb, status);
            used = 0;
          }
        }
        bits[s].consume(used);
        const uint32_t ra = __shfl_sync(0xffffffffu, rep[s], (int)sa);
        const uint32_t rb = __shfl_sync(0xffffffffu, rep[s], (int)sb);
        x[2 * h] = __fadd_rn(x[2 * h], __uint_as_float(ra));
        x[2 * h + 1] = __fadd_rn(x[2 * h + 1], __uint_as_float(rb));
      }
    }
    *reinterpret_cast<float4*>(out + i) = make_float4(x[0], x[1], x[2], x[3]);
  }
}

// Any other chunk (the ragged last one, or one too large for the staging areas): element by element from global
// memory with the canonical search; plain code, no warp votes.
struct GlobalChunk {
  const uint32_t* g[4];
  uint32_t nw[4];
  uint32_t start[4];
};
__device__ __noinline__ uint2 decode_any(const PairAux& A, const uint32_t* g, uint32_t nw, uint32_t bitpos,
                                         int32_t* status) {
  if (A.nused < 2) return make_uint2(A.rep[A.only_sym], 0u);
  auto rd = [&](uint32_t i) { return i < nw ? __ldg(g + i) : 0u; };
  const uint32_t wi = bitpos >> 5, p = bitpos & 31;
  const unsigned long long a = ((unsigned long long)rd(wi) << 32) | rd(wi + 1);
  const unsigned long long b = rd(wi + 2);
  const unsigned long long window = p ? ((a << p) | (b >> (32 - p))) : a;
  for (uint32_t L = 1; L <= A.max_len; ++L) {
    const unsigned long long c = window >> (64 - L);
    if (c >= A.first_code[L] && c - A.first_code[L] < A.len_count[L])
      return make_uint2(A.rep[A.sorted_sym[A.len_offset[L] + (uint32_t)(c - A.first_code[L])]], L);
  }
  set_status(status, LC_ERR_FORMAT);  // no code matches: damaged payload
  return make_uint2(0u, A.max_len);
}
template <int KS>
__device__ __noinline__ void decode_chunk_global(const PairStream* S, GlobalChunk G, const float* base, float* out,
                                                 uint64_t c, uint64_t n, uint32_t lane, int32_t* status) {
  uint32_t pos[KS];
#pragma unroll
  for (int s = 0; s < KS; ++s) pos[s] = G.start[s];
  for (uint32_t j = 0; j < kSteps; ++j) {
    for (uint32_t e = 0; e < kGroup; ++e) {
      const uint64_t i = c * kChunkElems + 128ull * j + 4 * lane + e;
      if (i >= n) continue;
      float x = base[i];
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        const uint2 ent = decode_any(S[s].aux, G.g[s], G.nw[s], pos[s], status);
        x = __fadd_rn(x, __uint_as_float(ent.x));
        pos[s] += ent.y;
      }
      out[i] = x;
    }
  }
}

// stage_bytes: bytes of staging area per warp and stream (a multiple of 16, at least 32).
template <int KS>
__global__ void __launch_bounds__(kDecMaxThreads, 1)
decode_pairs_kernel(const float* base, DecodeStreams streams, uint64_t n, float* out, int32_t* __restrict__ status,
                    const PairStream* __restrict__ tables, const uint32_t* __restrict__ flags, uint32_t stage_bytes) {
  // dynamic shared memory: [tables of the KS streams | staging areas | padding]
  extern __shared__ __align__(16) unsigned char s_raw[];
  if (*flags != 0) return;  // a stream was rejected, or this call belongs to the general decoder (same for all threads)
  PairStream* S = reinterpret_cast<PairStream*>(s_raw);
  {
    const uint4* src = reinterpret_cast<const uint4*>(tables);
    uint4* dst = reinterpret_cast<uint4*>(S);
    for (uint32_t i = threadIdx.x; i < KS * sizeof(PairStream) / 16; i += blockDim.x) dst[i] = __ldg(src + i);
  }
  __syncthreads();

  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
  unsigned char* stage0 = reinterpret_cast<unsigned char*>(S + KS) + (size_t)warp * KS * stage_bytes;
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  const uint64_t warp0 = (uint64_t)blockIdx.x * warps + warp;
  const uint64_t nwarps = (uint64_t)gridDim.x * warps;
  uint32_t rep[KS];  // lane j holds representative j of every stream
#pragma unroll
  for (int s = 0; s < KS; ++s) rep[s] = S[s].aux.rep[lane];

  for (uint64_t c = warp0; c < nchunks; c += nwarps) {
    Source W[KS];
    uint32_t start[KS], bytes[KS];
    unsigned long long off0[KS], off1[KS];
    bool fits = true;
    __syncwarp();  // the previous chunk's reads of the staging area are done
    // all index loads of all streams first, so that their latencies overlap
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint8_t* sp = streams.ptr[s];
      const unsigned long long* ci = reinterpret_cast<const unsigned long long*>(sp + S[s].aux.chunk_index_off);
      off0[s] = __ldg(ci + c);
      off1[s] = __ldg(ci + c + 1);
      const uint16_t* li = reinterpret_cast<const uint16_t*>(sp + S[s].aux.lane_index_off);
      start[s] = __ldg(li + c * kLanes + lane);
    }
    // then the asynchronous copies of the payloads into the staging areas
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      if (off0[s] > off1[s] || off1[s] > S[s].aux.payload_size || (off0[s] & 15) || (off1[s] & 15)) {
        set_status(status, LC_ERR_FORMAT);
        off0[s] = off1[s] = 0;
      }
      bytes[s] = (uint32_t)min(off1[s] - off0[s], (unsigned long long)kChunkElems * 8);
      const uint8_t* g = streams.ptr[s] + S[s].aux.payload_off + off0[s];
      unsigned char* st = stage0 + (size_t)s * stage_bytes;
      W[s].g = reinterpret_cast<const uint32_t*>(g);
      W[s].nw = bytes[s] >> 2;
      W[s].sbase = smem_addr(st);
      W[s].slim = W[s].sbase + bytes[s] + 12;
      // 16 bytes of zero slack after the chunk must fit too
      if (bytes[s] + 16 <= stage_bytes) {
        for (uint32_t k = lane * 16; k < bytes[s]; k += 32 * 16) cp_async_16(W[s].sbase + k, g + k);
        if (lane == 0) *reinterpret_cast<uint4*>(st + bytes[s]) = make_uint4(0, 0, 0, 0);
      } else {
        fits = false;
      }
    }
    cp_async_commit();
    // lane start offsets (exclusive scan of the lane bit counts) while the copies are in flight
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint32_t lane_bits = start[s];
      uint32_t incl = lane_bits;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
        if ((int)lane >= d) incl += v;
      }
      start[s] = min(incl - lane_bits, bytes[s] * 8u);
    }
    cp_async_wait_all();
    __syncwarp();
    if ((c + 1) * kChunkElems <= n && fits) {
      decode_chunk_pairs<KS>(S, W, start, rep, base, out, c, lane, status);
    } else {
      GlobalChunk G;
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        G.g[s] = W[s].g;
        G.nw[s] = W[s].nw;
        G.start[s] = start[s];
      }
      decode_chunk_global<KS>(S, G, base, out, c, n, lane, status);
    }
  }
}

template <int KS>
cudaError_t launch_pairs_ks(const float* base, const DecodeStreams& streams, uint64_t n, float* out, int32_t* status,
                            const PairStream* tables, const uint32_t* flags, cudaStream_t cs) {
  static int sms_of[kMaxDevices] = {};  // by device ordinal; non-zero once the kernel's attributes are set there
  constexpr uint32_t kTables = KS * sizeof(PairStream);
  constexpr uint32_t kMaxDyn = kSmemPerSm - 1024 - kOverrunBytes;  // room for static __shared__ and the padding
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  if (sms_of[dev] == 0) {
    int v = 0;
    cudaError_t e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_pairs_kernel<KS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(kMaxDyn + kOverrunBytes));
    if (e != cudaSuccess) return e;
    sms_of[dev] = v;
  }
  const int sms = sms_of[dev];
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  // Staging per warp and stream: 1.03 x the largest average chunk of the streams (from the buffer sizes, which
  // bound the payload). Among CTAs of 16, 12 and 8 warps, take the shape that puts most warps on an SM.
  uint64_t avg = 0;
  for (int s = 0; s < KS; ++s) {
    const uint64_t index_bytes = 72 * nchunks;  // lane and chunk index entries are not staged
    const uint64_t a = (streams.bytes[s] > index_bytes ? streams.bytes[s] - index_bytes : 0) / (nchunks ? nchunks : 1);
    avg = a > avg ? a : avg;
  }
  uint64_t want_stage = align_up(avg + avg / 32 + 48, 16);
  const uint64_t max_stage = kChunkElems * 5 / 8 + 16 + 16;  // five bits per element at most, padding, zero slack
  if (want_stage > max_stage) want_stage = max_stage;
  uint32_t warps = 8, stage = 0, dyn = 0, best_warps_per_sm = 0, ctas_per_sm = 1;
  for (uint32_t w = 16; w >= 8; w -= 4) {
    uint32_t st = (uint32_t)want_stage;
    if (kTables + (uint64_t)w * KS * st > kMaxDyn) {
      if (w > 8) continue;                               // try fewer warps first
      st = ((kMaxDyn - kTables) / (w * KS)) / 16 * 16;   // last resort: what fits; large chunks decode from global
    }
    const uint32_t d = kTables + w * KS * st + kOverrunBytes;
    int bps = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, decode_pairs_kernel<KS>, (int)(w * 32), d) != cudaSuccess)
      return cudaErrorUnknown;
    if (bps < 1) continue;
    if ((uint32_t)bps * w > best_warps_per_sm) {
      best_warps_per_sm = (uint32_t)bps * w;
      warps = w;
      stage = st;
      dyn = d;
      ctas_per_sm = (uint32_t)bps;
    }
  }
  if (best_warps_per_sm == 0) return cudaErrorLaunchOutOfResources;
  // chunk sizes vary around the average: give the staging areas whatever shared memory this shape leaves
  {
    const uint32_t budget = kSmemPerSm / ctas_per_sm - 1024 - 64;
    if (budget > kTables + kOverrunBytes) {
      uint32_t st = ((budget - kTables - kOverrunBytes) / (warps * KS)) / 16 * 16;
      if (st > max_stage) st = (uint32_t)max_stage;
      const uint32_t d = kTables + warps * KS * st + kOverrunBytes;
      int bps = 0;
      if (st > stage && d <= kMaxDyn + kOverrunBytes &&
          cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, decode_pairs_kernel<KS>, (int)(warps * 32), d) == cudaSuccess &&
          (uint32_t)bps >= ctas_per_sm) {
        stage = st;
        dyn = d;
      }
    }
  }
  uint64_t want = (nchunks + warps - 1) / warps;
  if (want == 0) return cudaSuccess;  // nothing to decode; the prepare kernel has validated the streams
  const uint64_t full = (uint64_t)sms * ctas_per_sm;
  const unsigned grid = (unsigned)(want < full ? want : full);
  {
    // shared-memory carve-out in percent of the SM's 228 KB: what the resident CTAs use (dynamic, static and the
    // 1 KB per CTA that the system reserves), so that whatever is left serves as L1
    int carve = (int)(((uint64_t)ctas_per_sm * (dyn + 2048) * 100 + 228 * 1024 - 1) / (228 * 1024)) + 1;
    if (carve > 100) carve = 100;
    if (cudaFuncSetAttribute(decode_pairs_kernel<KS>, cudaFuncAttributePreferredSharedMemoryCarveout, carve) != cudaSuccess)
      return cudaErrorUnknown;
  }
  decode_pairs_kernel<KS><<<grid, warps * 32, dyn, cs>>>(base, streams, n, out, status, tables, flags, stage);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_prepare(const DecodeStreams& streams, int k, uint64_t n, void* tables, uint32_t* flags,
                                  int32_t* status, cudaStream_t cs) {
  decode_prepare_kernel<<<k, kPrepThreads, 0, cs>>>(streams, n, static_cast<PairStream*>(tables), flags, status);
  return cudaGetLastError();
}

cudaError_t launch_decode_pairs(const float* base, const DecodeStreams& streams, int k, uint64_t n, float* out,
                                int32_t* status, const void* tables, const uint32_t* flags, cudaStream_t cs) {
  const PairStream* t = static_cast<const PairStream*>(tables);
  switch (k) {
    case 1: return launch_pairs_ks<1>(base, streams, n, out, status, t, flags, cs);
    case 2: return launch_pairs_ks<2>(base, streams, n, out, status, t, flags, cs);
    case 3: return launch_pairs_ks<3>(base, streams, n, out, status, t, flags, cs);
    case 4: return launch_pairs_ks<4>(base, streams, n, out, status, t, flags, cs);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace lc
