// Recovery pass: chunk-parallel Huffman decode of up to four streams fused with the chain add.
//
// Paper: the reconstruction identity u_t = u_0 + sum of the quantized deltas (Section 3, after
// component C2) and Algorithm 1 step 7 (tracked state += quantized delta), applied k times left to
// right in fp32. Stream layout: format text sections 2-4.
//
// One warp decodes one chunk; lane t walks lane sub-stream t of every stream at once, so at step j
// the warp holds 128 consecutive elements: one coalesced 16-byte load of base and one 16-byte store of
// out per lane, with the k representatives added in registers in between.
//
//  * The chunk's payload of every stream is first copied, coalesced, into a warp-private staging
//    area in shared memory; the lanes then pull their words from there. (Reading them straight from
//    global memory makes every refill touch one cache line per lane.) A chunk that does not fit the
//    staging area is decoded from global memory by the same code.
//  * Codes are looked up in shared-memory tables whose entries hold the representative itself. The
//    first level is indexed by the next kL1Bits bits and replicated 16 times (entry for (index, lane)
//    at index*16 + lane%16): a 64-bit shared load is served half a warp at a time, so the 16 lanes of
//    a half-warp always hit 16 different bank pairs although their indices are data dependent.
//    An entry whose 6-bit prefix belongs to longer codes points to a 64-entry sub-table indexed by the
//    next 6 bits (one predicated load, no branch), which resolves codes of up to 12 bits; still longer
//    codes are found by a canonical search behind a warp vote.
//  * A lane keeps a 64-bit bit buffer per stream and tops it up with one predicated word load before
//    every second symbol; that is enough because two table-resolved codes use at most 2*12 <= 33
//    bits.
//
// Every read of a stream is bounds-checked against the caller's buffer size and every table is
// validated before use, so a damaged stream yields LC_ERR_FORMAT (and unspecified output), never an
// out-of-bounds access.
//
// Bound: HBM at k = 1 (8 bytes per element + the stream); at k = 4 the integer work per symbol is
// the limit.
#include "lc_decode_bits.cuh"

namespace lc {
namespace {

using namespace dec;

constexpr int kDecMaxThreads = 512;
constexpr int kL1Bits = 6;
constexpr int kL1Rep = 16;
// Second level: one sub-table per 6-bit prefix that belongs to longer codes, all of one depth: the next 10 bits if a
// single prefix needs one (8 KB hold one table of 1024 entries; a Huffman code's long codes usually hang under one
// prefix), down to the next 4 bits if every prefix does (64 tables of 16 entries).
constexpr int kSubBitsMax = 10;
constexpr int kSubBitsMin = 4;
constexpr int kL2Bits = kL1Bits + kSubBitsMax;     // longest code the two table levels resolve
static_assert(kL2Bits <= 16, "the second code of a pair is looked up in the 32-bit upper word behind the first");
static_assert(((1 << kL1Bits) << (kSubBitsMin + 3)) <= 8192, "at the smallest depth every prefix gets a sub-table");
// Length field of a table entry that does not resolve its code. As a length it takes the bit count far below zero,
// which is how the hot loop notices: a step subtracts at most four of them per stream, and 1..4 times 2^29 (less a
// few real lengths) leaves the sign bit of the 32-bit count set in every case.
constexpr uint32_t kLongCode = 0x20000000u;
// distance, in steps of 512 bytes per warp, of the L2 prefetch of base (measured: 4, 6, 8, 12 and 16 rows; chains of
// two and more do not care between 4 and 12, a single stream is fastest at 6)
template <int KS>
constexpr int kPrefetchRows = KS == 1 ? 6 : 8;

// The two lookup tables of a stream are 8 KB each; the first starts on a 128-byte boundary of shared memory.
constexpr uint32_t kTableBytes = 8192;
constexpr uint32_t kTablePad = 128;  // the tables start on a 128-byte boundary (a lane's copy of an entry is chosen by OR)
static_assert((1 << kL1Bits) * kL1Rep * 8 == kTableBytes, "table sizes");

struct alignas(16) StreamState {
  uint2* l1;  // [(1 << kL1Bits) * kL1Rep] {bit pattern of rep, code length}; length kLongCode = not resolved here
  uint2* sub; // 8 KB of sub-tables of (1 << sub_bits) entries: {rep, length} or length kLongCode = longer code
  uint32_t sorted_rep[kMaxSymbols];   // representatives in canonical (len, id) order
  unsigned long long first_code[64];  // first canonical code of each length
  unsigned long long last_aligned[64]; // largest left-aligned 64-bit window whose code has at most this length
  uint32_t len_count[64];             // codes of each length
  uint32_t len_offset[64];            // index of the first of them in sorted_rep
  // header
  unsigned long long n, payload_bits, total_bytes, payload_off, payload_size;
  unsigned long long chunk_index_off, lane_index_off;
  uint32_t nsym, max_len, nchunks, only_rep;
  uint32_t fixed;  // fixed-width codes (format section 1.5): every symbol is coded, used or not
  uint32_t shared_table;  // the table comes from a larger vector (format section 1.6): unused symbols may have codes
  // validation accumulators
  unsigned long long kraft, count_sum, bit_sum;
  uint32_t seen_max, nused, nsub;
  uint32_t sub_bits;  // depth of the sub-tables, kSubBitsMin..kSubBitsMax: as many as 8 KB hold at that depth
  uint8_t sub_of_prefix[1 << kL1Bits], prefix_of_sub[1 << kL1Bits];
  uint8_t sym_len[kMaxSymbols];  // code length by symbol id
  uint32_t miss_count[2];  // first-level prefixes without a short code, per warp of 32 prefixes
  alignas(16) uint8_t hdr[kHeaderBytes];  // the stream header, staged
};

static_assert(sizeof(StreamState) % 16 == 0, "the staging areas behind the tables take 16-byte accesses");

// Canonical decode of the top `width` bits `idx`: (index into sorted_rep, length) or length 0 if the code
// is longer than `width`.
__device__ __forceinline__ uint2 canonical_lookup(const StreamState& S, uint32_t idx, uint32_t width) {
  for (uint32_t L = 1; L <= width; ++L) {
    const unsigned long long c = idx >> (width - L);
    if (c >= S.first_code[L] && c - S.first_code[L] < S.len_count[L])
      return make_uint2(S.len_offset[L] + (uint32_t)(c - S.first_code[L]), L);
  }
  return make_uint2(0u, 0u);
}

// Parses and validates stream `s`, then builds its decode tables in shared memory. All threads of the
// CTA call this; returns 0 or the error to report.
__device__ __noinline__ int prepare_stream(StreamState& S, unsigned char* tables, const uint8_t* __restrict__ s,
                              uint64_t bytes, uint64_t n, int* s_err) {
  const int tid = threadIdx.x, nthreads = blockDim.x;
  if (tid < 4 && bytes >= kHeaderBytes)
    reinterpret_cast<uint4*>(S.hdr)[tid] = __ldg(reinterpret_cast<const uint4*>(s) + tid);
  __syncthreads();
  if (tid == 0) {
    int err = 0;
    const uint8_t* h = S.hdr;
    S.l1 = reinterpret_cast<uint2*>(tables);
    S.sub = reinterpret_cast<uint2*>(tables + kTableBytes);
    S.kraft = 0; S.count_sum = 0; S.bit_sum = 0; S.seen_max = 0; S.nused = 0; S.only_rep = 0;
    if (bytes < kHeaderBytes) {
      err = LC_ERR_FORMAT;
    } else {
      const uint32_t nbits = h[6];
      S.n = load_le(h + 8, 8);
      S.nsym = (uint32_t)load_le(h + 16, 4);
      S.max_len = (uint32_t)load_le(h + 20, 4);
      S.nchunks = (uint32_t)load_le(h + 32, 4);
      S.payload_bits = load_le(h + 40, 8);
      S.total_bytes = load_le(h + 48, 8);
      S.payload_off = load_le(h + 56, 8);
      const bool magic = h[0] == 'L' && h[1] == 'C' && h[2] == 'C' && h[3] == '1';
      S.fixed = h[7] & 1u;
      S.shared_table = (h[7] >> 1) & 1u;
      if (!magic || load_le(h + 4, 2) != 1 || nbits < 1 || nbits > (uint32_t)kMaxNbits || (h[7] > 4 && h[7] != 8)) err = LC_ERR_FORMAT;  // bits 2 (cached lengths) and 3 (mean) go alone
      else if (S.nsym < 1 || S.nsym > (1u << nbits) || S.max_len > 63) err = LC_ERR_FORMAT;
      else if (load_le(h + 24, 4) != kChunkElems || load_le(h + 28, 2) != kLanes ||
               load_le(h + 30, 2) != kGroup || load_le(h + 36, 4) != kPayloadAlign) err = LC_ERR_FORMAT;
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
  for (int L = tid; L < 64; L += nthreads) S.len_count[L] = 0;
  __syncthreads();
  if (*s_err) return *s_err;

  // ---- table entries: a thread per symbol (up to 509 symbols, CTAs of 256 threads and more)
  const uint32_t nsym = S.nsym;
  const bool fixed = S.fixed != 0, shared_table = S.shared_table != 0;
  uint32_t fixed_width = 0;
  while ((1u << fixed_width) < nsym) fixed_width += 1;
  bool entry_bad = false;
  for (uint32_t sym = tid; sym < nsym; sym += nthreads) {
    const uint4 e = __ldg(reinterpret_cast<const uint4*>(s + kHeaderBytes) + sym);  // key:16 len:8 pad:8 | rep | count
    const uint32_t my_len = (e.x >> 16) & 255u, my_rep = e.y;
    const unsigned long long my_count = ((unsigned long long)e.w << 32) | e.z;
    entry_bad |= (e.x >> 24) != 0 || my_len > 63;
    entry_bad |= fixed ? (my_len != fixed_width) : (!shared_table && my_count == 0 && my_len != 0);
    entry_bad |= my_count != 0 && my_len == 0 && shared_table && S.max_len != 0;  // a used symbol needs its code
    S.sym_len[sym] = (uint8_t)my_len;
    atomicMax(&S.seen_max, my_len);
    if (my_count != 0) {
      atomicAdd(&S.count_sum, my_count);
      atomicAdd(&S.bit_sum, my_count * my_len);
    }
    if (!fixed && my_count != 0) S.only_rep = my_rep;  // meaningful only when no symbol has a code length
    if (fixed ? (fixed_width > 0 || sym == 0) : (shared_table && S.max_len != 0 ? my_len != 0 : my_count != 0)) {
      // the symbols that have a code
      atomicAdd(&S.nused, 1u);
      if (fixed && sym == 0) S.only_rep = my_rep;
      if (my_len > 0 && my_len <= 63) {
        atomicAdd(&S.kraft, 1ull << (63 - my_len));
        atomicAdd(&S.len_count[my_len], 1u);
      }
    }
  }
  if (__syncthreads_or(entry_bad)) return LC_ERR_FORMAT;
  if (tid == 0) {
    int err = 0;
    if (S.count_sum != S.n || S.bit_sum != S.payload_bits) err = LC_ERR_FORMAT;
    if (S.fixed) {
      uint32_t width = 0;
      while ((1u << width) < S.nsym) width += 1;
      if (S.max_len != width) err = LC_ERR_FORMAT;  // every entry's length was compared with the width above
    } else {
      if (S.seen_max != S.max_len) err = LC_ERR_FORMAT;
      if (S.nused >= 2) {
        if (S.kraft != (1ull << 63)) err = LC_ERR_FORMAT;
      } else if (S.max_len != 0) {
        err = LC_ERR_FORMAT;
      }
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
    // codes of length <= L fill the left-aligned range [0, (first_code[L] + count[L]) << (64 - L))
    for (int L = 1; L < 64; ++L) {
      const unsigned long long end = (S.first_code[L] + S.len_count[L]) << (64 - L);  // 0 when the range is everything
      S.last_aligned[L] = end - 1;
    }
    *s_err = err;
  }
  __syncthreads();
  if (*s_err) return *s_err;
  if (S.nused >= 2) {
    for (uint32_t sym = tid; sym < nsym; sym += nthreads) {
      const uint32_t my_len = S.sym_len[sym];
      if (my_len == 0) continue;  // a symbol without a code (unused, in a Huffman-coded stream)
      // rank among the symbols of the same length with smaller id
      uint32_t r = 0;
      for (uint32_t j = 0; j < sym; ++j) r += (S.sym_len[j] == my_len) ? 1u : 0u;
      S.sorted_rep[S.len_offset[my_len] + r] = __ldg(reinterpret_cast<const uint32_t*>(s + kHeaderBytes + 16 * sym + 4));
    }
  }
  if (S.nused < 2 && tid == 0) S.sorted_rep[0] = S.only_rep;
  __syncthreads();

  // ---- lookup tables: canonical decode of each entry's own index
  // First-level prefixes that belong to longer codes get a sub-table each. Sub-tables are as deep as
  // their number allows (8 KB in all).
  {
    const bool miss = tid < (1 << kL1Bits) && S.nused >= 2 && canonical_lookup(S, tid, kL1Bits).y == 0;
    const uint32_t ballot = __ballot_sync(0xffffffffu, miss);
    if (tid < (1 << kL1Bits) && (tid & 31) == 0) S.miss_count[tid >> 5] = __popc(ballot);
    __syncthreads();
    if (tid < (1 << kL1Bits)) {
      const uint32_t misses = S.miss_count[0] + S.miss_count[1];
      uint32_t sub_bits = kSubBitsMax;
      while (sub_bits > kSubBitsMin && misses > (kTableBytes >> (sub_bits + 3))) sub_bits -= 1;
      const uint32_t usable = kTableBytes >> (sub_bits + 3);  // >= misses: every such prefix gets a table
      const uint32_t rank = __popc(ballot & ((1u << (tid & 31)) - 1)) + (tid >= 32 ? S.miss_count[0] : 0u);
      uint32_t sub = 0;
      if (miss && rank < usable) {
        sub = rank;
        S.prefix_of_sub[sub] = (uint8_t)tid;
      }
      S.sub_of_prefix[tid] = (uint8_t)sub;
      if (tid == 0) {
        S.nsub = misses < usable ? misses : usable;
        S.sub_bits = sub_bits;
      }
    }
  }
  __syncthreads();
  const uint32_t sub_bits = S.sub_bits;
  for (uint32_t k = tid; k < (1u << kL1Bits) * kL1Rep; k += nthreads) {
    const uint32_t idx = k / kL1Rep;
    uint2 ent;
    if (S.nused < 2) {
      ent = make_uint2(S.only_rep, 0u);
    } else {
      const uint2 r = canonical_lookup(S, idx, kL1Bits);
      if (r.y) ent = make_uint2(S.sorted_rep[r.x], r.y);
      // address of the prefix's sub-table, less the offset that the prefix bits add when the lookup indexes it
      // with prefix and sub-table bits together (32-bit wrap-around arithmetic)
      else ent = make_uint2(smem_addr(S.sub) + ((uint32_t)S.sub_of_prefix[idx] << (sub_bits + 3)) -
                                ((idx << sub_bits) << 3), kLongCode);
    }
    S.l1[k] = ent;
  }
  for (uint32_t k = tid; k < kTableBytes / 8; k += nthreads) {
    const uint32_t sub = k >> sub_bits, j = k & ((1u << sub_bits) - 1);
    uint2 ent = make_uint2(0u, kLongCode);
    if (sub < S.nsub) {
      const uint2 r = canonical_lookup(S, ((uint32_t)S.prefix_of_sub[sub] << sub_bits) | j, kL1Bits + sub_bits);
      if (r.y) ent = make_uint2(S.sorted_rep[r.x], r.y);
    }
    S.sub[k] = ent;
  }
  __syncthreads();
  return 0;
}

// What the prepare kernel leaves in global memory for one stream and every CTA of the decode kernel copies: the two
// lookup tables, the stream's state, and the outcome of the validation. First-level entries that point to a sub-table
// hold that table's offset from the start of the sub-table area there (the shared address is added by the copy).
struct DecodeImage {
  uint2 l1[kTableBytes / 8];
  uint2 sub[kTableBytes / 8];
  StreamState state;
  int32_t err;
  int32_t pad_[3];
};
static_assert(sizeof(DecodeImage) <= kDecodeImageBytes, "the workspace region holds four of these");
static_assert(sizeof(DecodeImage) % 16 == 0 && sizeof(StreamState) % 16 == 0, "copied with 16-byte accesses");

constexpr int kPrepThreads = 512;
constexpr uint32_t kPrepSmem = kTableBytes + 2 * kTableBytes + sizeof(StreamState);

// One CTA per stream: parse, validate, build the tables (in this CTA's shared memory, as the decode kernel would),
// then write the image.
__global__ void __launch_bounds__(kPrepThreads)
decode_prepare_kernel(DecodeStreams streams, uint64_t n, DecodeImage* __restrict__ images) {
  extern __shared__ __align__(16) unsigned char p_raw[];
  unsigned char* tables = p_raw + ((kTableBytes - (smem_addr(p_raw) & (kTableBytes - 1))) & (kTableBytes - 1));
  StreamState& S = *reinterpret_cast<StreamState*>(p_raw + kTableBytes + 2 * kTableBytes);
  __shared__ int s_err;
  DecodeImage& img = images[blockIdx.x];
  const int err = prepare_stream(S, tables, streams.ptr[blockIdx.x], streams.bytes[blockIdx.x], n, &s_err);
  if (threadIdx.x == 0) img.err = err;
  if (err) return;
  const uint32_t sub_addr = smem_addr(S.sub);
  for (uint32_t k = threadIdx.x; k < kTableBytes / 8; k += kPrepThreads) {
    uint2 e = S.l1[k];
    if (e.y == kLongCode) e.x -= sub_addr;
    img.l1[k] = e;
    img.sub[k] = S.sub[k];
  }
  const uint4* src = reinterpret_cast<const uint4*>(&S);
  uint4* dst = reinterpret_cast<uint4*>(&img.state);
  for (uint32_t k = threadIdx.x; k < sizeof(StreamState) / 16; k += kPrepThreads) dst[k] = src[k];
}

// Two-level table lookup of the code at the top of `hi`: {representative, length}, length kLongCode if
// the tables do not resolve it. `l1lane` = shared address of this lane's copy of first-level entry 0.
// The first-level entry of a prefix that belongs to longer codes holds the shared address of the
// prefix's sub-table, which is read by a predicated load (no branch for the few lanes that need it).
// Written in PTX so that index scaling and base addition stay multiply-adds (they then run beside the
// shifts and compares instead of competing with them for the integer pipe).
template <int OFFSET>
__device__ __forceinline__ uint2 lookup_code(uint32_t hi, uint32_t l1lane, uint32_t sub_shift) {
  uint2 ent;
  asm("{\n\t"
      ".reg .u32 t, a;\n\t"
      ".reg .pred q;\n\t"
      "shr.u32 t, %2, %4;\n\t"
      "mad.lo.u32 a, t, %5, %3;\n\t"
      "ld.shared.v2.u32 {%0,%1}, [a+%8];\n\t"
      "setp.gt.u32 q, %1, 63;\n\t"
      "shr.u32 t, %2, %7;\n\t"         // prefix and sub-table index together: the entry's address allows for the prefix
      "mad.lo.u32 a, t, 8, %0;\n\t"
      "@q ld.shared.v2.u32 {%0,%1}, [a];\n\t"
      "}"
      : "=&r"(ent.x), "=&r"(ent.y)
      : "r"(hi), "r"(l1lane), "n"(32 - kL1Bits), "n"(kL1Rep * 8), "n"(kL1Bits), "r"(sub_shift), "n"(OFFSET));
  return ent;
}

// Code the tables did not resolve: canonical search on a 64-bit window read from the chunk, then re-seat
// the lane's bit buffer behind the code. Returns the representative.
template <bool STAGED>
__device__ __forceinline__ uint32_t long_code(LaneBits<STAGED>& B, const StreamState& S, const Source& W,
                                              int32_t* status) {
  const uint32_t pos = B.bitpos(W);
  const uint32_t idx = pos >> 5, sh = pos & 31;
  const uint32_t w0 = B.word(W, idx), w1 = B.word(W, idx + 1), w2 = B.word(W, idx + 2);
  const unsigned long long window =
      ((unsigned long long)__funnelshift_l(w1, w0, sh) << 32) | __funnelshift_l(w2, w1, sh);
  // the first level resolves shorter codes, and so does the prefix's sub-table if it has a real one
  uint32_t L = kL1Bits + 1 + (S.sub_of_prefix[window >> (64 - kL1Bits)] < S.nsub ? S.sub_bits : 0u);
  while (L < S.max_len && (S.len_count[L] == 0 || window > S.last_aligned[L])) L += 1;
  const unsigned long long code = window >> (64 - L);
  uint32_t rep = 0;
  if (L <= S.max_len && code >= S.first_code[L] && code - S.first_code[L] < S.len_count[L]) {
    rep = S.sorted_rep[S.len_offset[L] + (uint32_t)(code - S.first_code[L])];
  } else {
    set_status(status, LC_ERR_FORMAT);  // no code matches: damaged payload
  }
  B.seek(W, pos + L);
  return rep;
}

// Full chunk: the hot loop. Per step a lane decodes 4 elements x KS streams; the KS streams are independent
// dependency chains and are written interleaved.
//
// The loop body is straight-line code. A lane tops its bit buffers up once per step and then decodes its four
// codes per stream from the upper word alone, two at a time (the second lookup takes the first code's length,
// the buffer is shifted once per pair). Two things can go wrong for a lane in a step, both rare: a code longer
// than the tables resolve, and four codes that take more bits than the buffer held (32 are guaranteed, four
// table-resolved codes can take 64). Both show as a negative bit count at the end of the step: the marker of an
// unresolved code is a huge length, and a lookup on too few valid bits always overdraws, because no code is a
// prefix of another. One warp vote per step finds them, and the flagged lanes decode the step again from where it
// started, one code at a time with a top-up before each (a top-up makes 32 bits valid, a table-resolved code
// takes at most 16). Whatever the quick pass did to their buffers in
// between stays inside the staged chunk (a top-up moves one word per step) and is discarded.
template <int KS, bool STAGED>
__device__ __forceinline__ void decode_chunk_fast(const StreamState* S, const Source* W, const uint32_t* start,
                                                    const float* base, float* out, uint64_t c, uint32_t lane,
                                                    const float* next_rows, int32_t* status) {
  LaneBits<STAGED> bits[KS];
  // the streams' tables follow each other at 2 * kTableBytes: one base address, the rest as immediate offsets
  const uint32_t l1lane = smem_addr(S[0].l1) | ((lane & (kL1Rep - 1)) * 8u);
  uint32_t sub_shift[KS];
#pragma unroll
  for (int s = 0; s < KS; ++s) {
    bits[s].seek(W[s], start[s]);
    sub_shift[s] = 32 - kL1Bits - S[s].sub_bits;
  }
  const uint64_t e0 = c * kChunkElems + 4 * lane;
  float4 b = ldg_stream_v4(base + e0);
  // With one stream a step is short, and one row of base in registers ahead of its use leaves too few bytes in flight
  // for the L2's latency (0.80 of the copy rate); a second row brings that to 0.92. With two or more streams the
  // second row makes the kernel slower (measured for 2, 3 and 4 streams), so they keep one.
  float4 b2 = b;
  if (KS == 1) b2 = ldg_stream_v4(base + e0 + 128);
  // Rows of base are asked into the L2 kPrefetchRows steps before they are loaded: a warp has one row in
  // registers ahead of its use, which alone leaves far too few bytes in flight per SM for the DRAM latency.
  // Behind this chunk's last row the requests go on with the first rows of the chunk this warp decodes next
  // (`next_rows`: this lane's part of that chunk's first row, or of this chunk's first row if there is none).
  const float* pf = base + e0 + 128 * kPrefetchRows<KS>;
#pragma unroll 1
  for (uint32_t j = 0; j < kSteps; ++j) {
    const uint64_t i = e0 + 128ull * j;
    float x[4] = {b.x, b.y, b.z, b.w};
    // the 16 bytes of base of a later step, requested one step ahead (one stream: two steps); the last steps
    // re-read their own
    if (KS == 1) {
      b = b2;
      b2 = ldg_stream_v4(base + i + (j + 2 < kSteps ? 256 : 0));
    } else {
      b = ldg_stream_v4(base + i + (j + 1 < kSteps ? 128 : 0));
    }
    asm volatile("prefetch.global.L2 [%0];" ::"l"(pf));
    pf = (j == kSteps - kPrefetchRows<KS> - 1) ? next_rows : pf + 128;
    int cnt0[KS];
    uint32_t flags = 0;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      bits[s].refill(W[s]);
      cnt0[s] = bits[s].cnt;  // where the step starts, for the careful pass (`next` does not move within a step)
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint2 ea[KS], eb[KS];
      uint32_t h1[KS];
      ea[0] = lookup_code<0>(bits[0].hi, l1lane, sub_shift[0]);
      if (KS > 1) ea[1 % KS] = lookup_code<2 * kTableBytes>(bits[1 % KS].hi, l1lane, sub_shift[1 % KS]);
      if (KS > 2) ea[2 % KS] = lookup_code<4 * kTableBytes>(bits[2 % KS].hi, l1lane, sub_shift[2 % KS]);
      if (KS > 3) ea[3 % KS] = lookup_code<6 * kTableBytes>(bits[3 % KS].hi, l1lane, sub_shift[3 % KS]);
#pragma unroll
      for (int s = 0; s < KS; ++s) h1[s] = __funnelshift_l(0u, bits[s].hi, ea[s].y);  // hi << length (mod 32)
      eb[0] = lookup_code<0>(h1[0], l1lane, sub_shift[0]);
      if (KS > 1) eb[1 % KS] = lookup_code<2 * kTableBytes>(h1[1 % KS], l1lane, sub_shift[1 % KS]);
      if (KS > 2) eb[2 % KS] = lookup_code<4 * kTableBytes>(h1[2 % KS], l1lane, sub_shift[2 % KS]);
      if (KS > 3) eb[3 % KS] = lookup_code<6 * kTableBytes>(h1[3 % KS], l1lane, sub_shift[3 % KS]);
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        x[2 * h] = __fadd_rn(x[2 * h], __uint_as_float(ea[s].x));
        x[2 * h + 1] = __fadd_rn(x[2 * h + 1], __uint_as_float(eb[s].x));
        const uint32_t len = ea[s].y + eb[s].y;
        bits[s].hi = __funnelshift_l(bits[s].lo, bits[s].hi, len);
        bits[s].lo = __funnelshift_l(0u, bits[s].lo, len);
        bits[s].cnt = (int)((uint32_t)bits[s].cnt - len);
      }
    }
#pragma unroll
    for (int s = 0; s < KS; ++s) flags |= (uint32_t)bits[s].cnt;
    if (__builtin_expect(__any_sync(0xffffffffu, (int)flags < 0), 0)) {
      if ((int)flags < 0) {
        const float4 b0 = ldg_stream_v4(base + i);
        x[0] = b0.x; x[1] = b0.y; x[2] = b0.z; x[3] = b0.w;
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          bits[s].cnt = cnt0[s];
          bits[s].seek(W[s], bits[s].bitpos(W[s]));
        }
        // one element per trip; x is rotated so that the loop needs no indexed register
#pragma unroll 1
        for (int e = 0; e < 4; ++e) {
          float v = x[0];
          uint2 ent[KS];
#pragma unroll
          for (int s = 0; s < KS; ++s) bits[s].refill(W[s]);
          ent[0] = lookup_code<0>(bits[0].hi, l1lane, sub_shift[0]);
          if (KS > 1) ent[1 % KS] = lookup_code<2 * kTableBytes>(bits[1 % KS].hi, l1lane, sub_shift[1 % KS]);
          if (KS > 2) ent[2 % KS] = lookup_code<4 * kTableBytes>(bits[2 % KS].hi, l1lane, sub_shift[2 % KS]);
          if (KS > 3) ent[3 % KS] = lookup_code<6 * kTableBytes>(bits[3 % KS].hi, l1lane, sub_shift[3 % KS]);
#pragma unroll
          for (int s = 0; s < KS; ++s) {
            if (ent[s].y > 63u) ent[s] = make_uint2(long_code<STAGED>(bits[s], S[s], W[s], status), 0u);  // consumed
            v = __fadd_rn(v, __uint_as_float(ent[s].x));
            bits[s].consume(ent[s].y);
          }
          x[0] = x[1]; x[1] = x[2]; x[2] = x[3]; x[3] = v;
        }
      }
    }
    *reinterpret_cast<float4*>(out + i) = make_float4(x[0], x[1], x[2], x[3]);
  }
}
static_assert(kL1Rep * 8 == 128, "first-level entries of one index span 128 bytes");

// The vector's last, partial chunk: element by element (indices beyond n are skipped), each code with a top-up, a
// table lookup and, if the tables do not resolve it, the canonical search. Out of line: it runs once per call, in one
// warp, and must not weigh on the registers of the loop above. The chunk's words come from the staging areas if
// they fit there (a single warp waiting for global memory at every code would take several times as long as all the
// other chunks of a medium-sized vector together), else from global memory.
struct PartialChunk {
  Source W[4];
  uint32_t start[4];
  uint32_t sub_shift[4];
};
template <int KS, bool STAGED>
__device__ __noinline__ void decode_chunk_partial(const StreamState* S, PartialChunk P, uint32_t l1lane,
                                                  const float* base, float* out, uint64_t c, uint64_t n, uint32_t lane,
                                                  int32_t* status) {
  LaneBits<STAGED> bits[KS];
#pragma unroll
  for (int s = 0; s < KS; ++s) bits[s].seek(P.W[s], P.start[s]);
#pragma unroll 1
  for (uint32_t j = 0; j < kSteps; ++j) {
#pragma unroll 1
    for (uint32_t e = 0; e < kGroup; ++e) {
      const uint64_t i = c * kChunkElems + 128ull * j + 4 * lane + e;
      if (i >= n) continue;
      float x = base[i];
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        bits[s].refill(P.W[s]);
        uint2 ent = lookup_code<0>(bits[s].hi, l1lane + s * 2 * kTableBytes, P.sub_shift[s]);
        if (ent.y > 63u) ent = make_uint2(long_code<STAGED>(bits[s], S[s], P.W[s], status), 0u);  // consumed
        x = __fadd_rn(x, __uint_as_float(ent.x));
        bits[s].consume(ent.y);
      }
      out[i] = x;
    }
  }
}

// stage_bytes: bytes of staging area per warp and stream (a multiple of 16, at least 32).
template <int KS>
__global__ void __launch_bounds__(kDecMaxThreads, 1)
decode_kernel(const float* base, DecodeStreams streams, uint64_t n, float* out, int32_t* __restrict__ status,
              const DecodeImage* __restrict__ images, uint32_t stage_bytes, uint64_t chunk_begin, uint64_t chunk_end) {
  // dynamic shared memory: [pad to 128 bytes | 2 tables per stream | StreamState per stream | staging areas]
  extern __shared__ __align__(16) unsigned char s_raw[];
  unsigned char* tables = s_raw + ((kTablePad - (smem_addr(s_raw) & (kTablePad - 1))) & (kTablePad - 1));
  StreamState* S = reinterpret_cast<StreamState*>(s_raw + kTablePad + KS * 2 * kTableBytes);
  // A launch of a single CTA (a vector of a few chunks) validates the streams and builds their tables itself, which
  // saves the prepare kernel's launch; `images` is null then.
  __shared__ int s_err;
  if (images == nullptr) {
    for (int s = 0; s < KS; ++s) {
      const int err = prepare_stream(S[s], tables + s * 2 * kTableBytes, streams.ptr[s], streams.bytes[s], n, &s_err);
      if (err) {  // the same value for every thread
        if (threadIdx.x == 0) set_status(status, err);
        return;
      }
    }
  }
  // otherwise the streams were validated and their tables built by decode_prepare_kernel: report a rejected stream
  // (the same words for every thread) or copy the images in
#pragma unroll
  for (int s = 0; s < KS; ++s) {
    const int err = images ? images[s].err : 0;
    if (err) {
      if (threadIdx.x == 0) set_status(status, err);
      return;
    }
  }
#pragma unroll
  for (int s = 0; s < KS && images != nullptr; ++s) {
    uint2* l1 = reinterpret_cast<uint2*>(tables + s * 2 * kTableBytes);
    uint2* sub = l1 + kTableBytes / 8;
    const uint32_t sub_addr = smem_addr(sub);
    for (uint32_t k = threadIdx.x; k < kTableBytes / 8; k += blockDim.x) {
      uint2 e = __ldg(&images[s].l1[k]);
      if (e.y == kLongCode) e.x += sub_addr;
      l1[k] = e;
      sub[k] = __ldg(&images[s].sub[k]);
    }
    const uint4* src = reinterpret_cast<const uint4*>(&images[s].state);
    uint4* dst = reinterpret_cast<uint4*>(&S[s]);
    for (uint32_t k = threadIdx.x; k < sizeof(StreamState) / 16; k += blockDim.x) dst[k] = __ldg(src + k);
  }
  __syncthreads();
  if (threadIdx.x < KS) {
    S[threadIdx.x].l1 = reinterpret_cast<uint2*>(tables + threadIdx.x * 2 * kTableBytes);
    S[threadIdx.x].sub = S[threadIdx.x].l1 + kTableBytes / 8;
  }
  __syncthreads();

  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
  unsigned char* stage0 = reinterpret_cast<unsigned char*>(S + KS) + (size_t)warp * KS * stage_bytes;
  const uint64_t warp0 = chunk_begin + (uint64_t)blockIdx.x * warps + warp;  // this launch decodes [chunk_begin, chunk_end)
  const uint64_t nwarps = (uint64_t)gridDim.x * warps;

  for (uint64_t c = warp0; c < chunk_end; c += nwarps) {
    Source W[KS];
    uint32_t start[KS], bytes[KS];
    unsigned long long off0[KS], off1[KS];
    bool fits = true;
    __syncwarp();  // the previous chunk's reads of the staging area are done
    // all index loads of all streams first, so that their latencies overlap
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const uint8_t* sp = streams.ptr[s];
      const unsigned long long* ci = reinterpret_cast<const unsigned long long*>(sp + S[s].chunk_index_off);
      off0[s] = __ldg(ci + c);
      off1[s] = __ldg(ci + c + 1);
      const uint16_t* li = reinterpret_cast<const uint16_t*>(sp + S[s].lane_index_off);
      start[s] = __ldg(li + c * kLanes + lane);
    }
    // then the asynchronous copies of the payloads into the staging areas
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      if (off0[s] > off1[s] || off1[s] > S[s].payload_size || (off0[s] & 15) || (off1[s] & 15)) {
        set_status(status, LC_ERR_FORMAT);
        off0[s] = off1[s] = 0;
      }
      bytes[s] = (uint32_t)min(off1[s] - off0[s], (unsigned long long)kChunkElems * 8);
      const uint8_t* g = streams.ptr[s] + S[s].payload_off + off0[s];
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
    if ((c + 1) * kChunkElems <= n) {
      // where the L2 prefetch goes on behind this chunk: the next chunk of this warp, if it is a full one
      const uint64_t cn = c + nwarps;
      const float* next_rows = base + (cn < chunk_end && (cn + 1) * kChunkElems <= n ? cn : c) * kChunkElems + 4 * lane;
      if (fits) decode_chunk_fast<KS, true>(S, W, start, base, out, c, lane, next_rows, status);
      else decode_chunk_fast<KS, false>(S, W, start, base, out, c, lane, next_rows, status);
    } else {
      PartialChunk P;
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        P.W[s] = W[s];
        P.start[s] = start[s];
        P.sub_shift[s] = 32 - kL1Bits - S[s].sub_bits;
      }
      const uint32_t l1lane = smem_addr(S[0].l1) | ((lane & (kL1Rep - 1)) * 8u);
      if (fits) decode_chunk_partial<KS, true>(S, P, l1lane, base, out, c, n, lane, status);
      else decode_chunk_partial<KS, false>(S, P, l1lane, base, out, c, n, lane, status);
    }
  }
}

template <int KS>
cudaError_t launch_decode_ks(const float* base, const DecodeStreams& streams, uint64_t n, float* out,
                             int32_t* status, DecodeImage* images, uint64_t chunk_begin, uint64_t chunk_end,
                             bool prepare, cudaStream_t cs) {
  static int sms_of[kMaxDevices] = {};  // by device ordinal; non-zero once the kernel's attributes are set there
  constexpr uint32_t kTables = kTablePad + KS * (2 * kTableBytes + sizeof(StreamState));
  constexpr uint32_t kMaxDyn = kSmemPerSm - 1024 - kOverrunBytes;  // room for static __shared__ and the padding
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  if (sms_of[dev] == 0) {
    int v = 0;
    cudaError_t e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_kernel<KS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(kMaxDyn + kOverrunBytes));
    if (e != cudaSuccess) return e;
    sms_of[dev] = v;
  }
  const int sms = sms_of[dev];
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  // Staging per warp and stream: 1.03 x the largest average chunk of the streams (from the buffer sizes,
  // which bound the payload). Among CTAs of 16, 12 and 8 warps, take the shape that puts most warps on an
  // SM (shared memory and registers both count; with four streams that is one CTA of 16 warps, with one
  // stream several smaller CTAs).
  uint64_t avg = 0;
  for (int s = 0; s < KS; ++s) {
    const uint64_t index_bytes = 72 * nchunks;  // lane and chunk index entries are not staged
    const uint64_t a = (streams.bytes[s] > index_bytes ? streams.bytes[s] - index_bytes : 0) / (nchunks ? nchunks : 1);
    avg = a > avg ? a : avg;
  }
  uint64_t want_stage = align_up(avg + avg / 32 + 48, 16);
  if (want_stage > kChunkElems * 8 + 16) want_stage = kChunkElems * 8 + 16;
  uint32_t warps = 8, stage = 0, dyn = 0, best_warps_per_sm = 0, ctas_per_sm = 1;
  for (uint32_t w = 16; w >= 8; w -= 4) {
    uint32_t st = (uint32_t)want_stage;
    if (kTables + (uint64_t)w * KS * st > kMaxDyn) {
      if (w > 8) continue;                               // try fewer warps first
      st = ((kMaxDyn - kTables) / (w * KS)) / 16 * 16;   // last resort: what fits; large chunks decode from global
    }
    const uint32_t d = kTables + w * KS * st + kOverrunBytes;
    int bps = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, decode_kernel<KS>, (int)(w * 32), d) != cudaSuccess)
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
      if (st > kChunkElems * 8 + 16) st = kChunkElems * 8 + 16;
      const uint32_t d = kTables + warps * KS * st + kOverrunBytes;
      int bps = 0;
      if (st > stage && d <= kMaxDyn + kOverrunBytes &&
          cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, decode_kernel<KS>, (int)(warps * 32), d) == cudaSuccess &&
          (uint32_t)bps >= ctas_per_sm) {
        stage = st;
        dyn = d;
      }
    }
  }
  uint64_t want = (chunk_end - chunk_begin + warps - 1) / warps;
  if (want == 0) want = 1;  // still reports a rejected stream
  const uint64_t full = (uint64_t)sms * ctas_per_sm;
  const unsigned grid = (unsigned)(want < full ? want : full);
  {
    // shared-memory carve-out in percent of the SM's 228 KB: what the resident CTAs use (dynamic, static and the
    // 1 KB per CTA that the system reserves), so that whatever is left serves as L1
    int carve = (int)(((uint64_t)ctas_per_sm * (dyn + 2048) * 100 + 228 * 1024 - 1) / (228 * 1024)) + 1;
    if (carve > 100) carve = 100;
    if (cudaFuncSetAttribute(decode_kernel<KS>, cudaFuncAttributePreferredSharedMemoryCarveout, carve) != cudaSuccess)
      return cudaErrorUnknown;
  }
  // The streams' tables: built by one CTA per stream ahead of a launch of many CTAs, by the decoding CTA itself when
  // there is only one (`images` null), or left from an earlier launch over the same streams (`prepare` false).
  const DecodeImage* use = images;
  if (prepare) {
    if (grid == 1) {
      use = nullptr;
    } else {
      decode_prepare_kernel<<<KS, kPrepThreads, kPrepSmem, cs>>>(streams, n, images);
      if (cudaGetLastError() != cudaSuccess) return cudaErrorLaunchFailure;
    }
  }
  decode_kernel<KS><<<grid, warps * 32, dyn, cs>>>(base, streams, n, out, status, use, stage, chunk_begin, chunk_end);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode(const float* base, const DecodeStreams& streams, int k, uint64_t n, float* out,
                          int32_t* status, void* images, cudaStream_t cs, uint64_t chunk_begin, uint64_t chunk_end,
                          bool prepare) {
  if (k < 1 || k > 4) return cudaErrorInvalidValue;
  const uint64_t all_chunks = (n + kChunkElems - 1) / kChunkElems;
  if (chunk_end > all_chunks) chunk_end = all_chunks;
  if (chunk_begin > chunk_end) chunk_begin = chunk_end;
  static bool prep_ready[kMaxDevices] = {};  // by device ordinal
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  if (!prep_ready[dev]) {
    const cudaError_t e = cudaFuncSetAttribute(decode_prepare_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)kPrepSmem);
    if (e != cudaSuccess) return e;
    prep_ready[dev] = true;
  }
  DecodeImage* img = static_cast<DecodeImage*>(images);
  switch (k) {
    case 1: return launch_decode_ks<1>(base, streams, n, out, status, img, chunk_begin, chunk_end, prepare, cs);
    case 2: return launch_decode_ks<2>(base, streams, n, out, status, img, chunk_begin, chunk_end, prepare, cs);
    case 3: return launch_decode_ks<3>(base, streams, n, out, status, img, chunk_begin, chunk_end, prepare, cs);
    case 4: return launch_decode_ks<4>(base, streams, n, out, status, img, chunk_begin, chunk_end, prepare, cs);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace lc
