// Encode pass: key plane -> Huffman bitstream with chunk and lane indices.
//
// Paper: Algorithm 1 step 6 and Section 3.1.2 (the quantized delta, i.e. the sequence of bucket
// indices, is Huffman-coded). Element order, bit order and the two indices are those of the stream
// format text, sections 2 and 3.
//
// A CTA takes a tile of 8 consecutive chunks, one per warp; lane t owns lane sub-stream t. Per chunk:
//   A. every lane codes its 128 elements into its own column of a warp-private word matrix in shared
//      memory (word k of lane t at k*32 + t: plain stores, no bank conflicts, no atomics). Code and
//      length come packed in one 32-bit table entry (a 16-byte entry made the lookups saturate the
//      shared-memory pipe) and two neighbouring codes are appended as one; the rare codes of 17..32 bits
//      sit behind one vote per four elements. Emitting a finished word is a handful of predicated
//      instructions;
//   B. a warp shuffle scan of the lane bit counts gives every lane its bit offset in the chunk (the
//      lane index of the stream) and the chunk its size, which is published at once;
//   C. the lanes' words are shifted to their bit offsets and ORed into the chunk image (shared memory);
//   D. the tile's byte offset comes from an exclusive scan over all tiles, done across CTAs with a
//      decoupled look-back over per-tile descriptors (per-chunk descriptors were tried: with thousands
//      of chunks in flight every look-back walks too far back);
//   E. the chunk image is copied to the payload with coalesced 16-byte stores.
// The loop is software-pipelined: D and E of a tile run after A and B of the CTA's next tile (whose C follows
// once E has freed the image area), and D is done by whichever warp finishes coding first (see the loop). Tiles are handed out by an atomic ticket, so
// every tile a CTA waits for in D has already been started by a running CTA, and coding never waits for
// anything. The wait is bounded all the same: after `spin_limit` polls the CTA records LC_ERR_TIMEOUT, marks
// its tile aborted (successors see that at once and abort too) and moves on.
// A caller that wants no device-side wait at all selects the two-pass scan (EncodeOptions::two_pass_scan):
// encode_sizes_kernel computes every chunk's size, encode_scan_kernel (one CTA) turns the sizes into the chunk
// index, and this kernel takes its offsets from there instead of looking back. Same bytes, one more pass over
// the key plane.
//
// Rare cases take a compact two-pass path (lengths, then bits ORed in place): the ragged last chunk,
// codes longer than 32 bits, a lane or chunk that outgrows its shared-memory area, and vectors with an
// exponent field >= 128, for which the one-byte key plane is not enough and keys come from base and cur.
//
// Bound: reads 1 byte and writes about 0.5 bytes per element, so this pass is limited by the integer
// work per element, not by HBM.
#include "lc_common.cuh"

namespace lc {
namespace {

constexpr int kEncThreads = kEncWarps * 32;
// 48 KB of dynamic shared memory per CTA (four CTAs per SM), split evenly between the warps that work:
// all 8 while an average chunk fits half of a 6 KB share (column matrix + chunk image), else 4, 2 or 1.
constexpr uint32_t kEncSmem = 48 * 1024;
constexpr int kUpdRows = 4;  // rows of base in flight per warp in the kernel that also writes the tracked state
constexpr uint32_t kUpdSmem = kEncWarps * kUpdRows * 512;  // its ring, behind the kEncSmem bytes of coding areas
constexpr int kLookBack = 8;  // look-back sub-windows of 32 tile descriptors read per round

constexpr uint32_t kPackedLenShift = 26;                      // packed entry: length << 26 | code
constexpr uint32_t kPackedCodeMask = (1u << kPackedLenShift) - 1;
constexpr uint32_t kPackedMaxLen = 16;                        // two packed codes make one append of <= 32 bits
constexpr uint32_t kPackedLong = 63;                          // length field of a code that does not fit

struct Tables {
  uint32_t packed[256];  // by plane byte: length << 26 | code for codes of up to 16 bits, else length field 63
  uint2 full[256];       // by plane byte: {code, length} for codes of up to 32 bits
};

// Where the slow path gets an element's key from.
struct KeySource {
  const uint8_t* plane;  // used unless `wide`
  const float* base;
  const float* cur;
  bool wide;
  __device__ __forceinline__ uint32_t key(uint64_t c, uint32_t j, uint32_t lane, uint32_t e) const {
    if (wide) {
      const uint64_t i = c * kChunkElems + 128ull * j + 4 * lane + e;
      return __float_as_uint(__fsub_rn(cur[i], base[i])) >> 23;
    }
    const uint32_t b = plane[c * kChunkElems + (j >> 2) * 512 + lane * 16 + (j & 3) * 4 + e];
    return ((b & 1u) << 8) | (b >> 1);
  }
};

// Appends a code of at most 32 bits to the lane's bit accumulator and ORs completed 32-bit words into the
// chunk image at `dst` (shared or global memory).
struct OrPacker {
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

// Slow, compact path (see the header). With dst == nullptr it only returns the lane's bit count;
// otherwise it ORs the lane's bits into the zeroed chunk image at dst, starting at bit lane_start.
// The plane bytes of four steps are read as one 16-byte vector, the way the fast path reads them (this path also
// codes the vector's partial last chunk, alone in its warp). Codes come from the per-key table in global memory:
// passing the CTA's shared tables in as well was measured to cost the kernel's main loop 4 %.
__device__ __noinline__ uint32_t chunk_slow(const EncEntry* __restrict__ enc, KeySource ks, uint64_t c,
                                            uint32_t lane, uint64_t n, uint32_t* dst, uint32_t lane_start) {
  OrPacker pk{0ull, lane_start & 31u, dst ? dst + (lane_start >> 5) : nullptr};
  uint32_t bits = 0;
  const bool from_plane = !ks.wide;
  for (uint32_t q = 0; q < kSteps / 4; ++q) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (from_plane) v = __ldg(reinterpret_cast<const uint4*>(ks.plane + c * kChunkElems + q * 512) + lane);
    const uint32_t words[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (uint32_t r = 0; r < 4; ++r) {
      const uint32_t j = 4 * q + r;
#pragma unroll
      for (uint32_t e = 0; e < kGroup; ++e) {
        const uint64_t i = c * kChunkElems + 128ull * j + 4 * lane + e;
        if (i >= n) continue;
        uint32_t key;
        if (from_plane) {
          const uint32_t b = (words[r] >> (8 * e)) & 255u;
          key = ((b & 1u) << 8) | (b >> 1);
        } else {
          key = ks.key(c, j, lane, e);
        }
        const EncEntry en = enc[key];
        const uint32_t code_lo = en.code_lo, code_hi = en.code_hi, len = en.len;
        bits += len;
        if (dst) {
          if (len > 32) {
            pk.put(code_hi, len - 32);
            pk.put(code_lo, 32);
          } else {
            pk.put(code_lo, len);
          }
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

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Fast-path state of a lane: pending bits in hi:lo (low `nb` bits valid), next word slot in its column.
struct ColumnPacker {
  uint32_t hi, lo, nb;
  uint32_t dst;  // shared address of the next word of this lane's column (stride 128 bytes)
  uint32_t lim;  // shared address one past the column
  __device__ __forceinline__ void put(uint32_t code, uint32_t len) {
    // (hi:lo) = (hi:lo) << len | code, len <= 32
    hi = __funnelshift_lc(lo, hi, len);
    lo = __funnelshift_lc(0u, lo, len) | code;
    nb += len;
    // emit the oldest 32 pending bits once there are 32 or more, unless the column is full
    asm volatile(
        "{\n\t"
        ".reg .pred q;\n\t"
        ".reg .u32 w;\n\t"
        "setp.ge.u32 q, %0, 32;\n\t"
        "setp.lt.and.u32 q, %1, %4, q;\n\t"
        "@q sub.u32 %0, %0, 32;\n\t"
        "@q shf.r.clamp.b32 w, %3, %2, %0;\n\t"
        "@q st.shared.u32 [%1], w;\n\t"
        "@q add.u32 %1, %1, 128;\n\t"
        "}"
        : "+r"(nb), "+r"(dst)
        : "r"(hi), "r"(lo), "r"(lim)
        : "memory");
  }
};

// UPDATE: the kernel also writes the tracked state of Algorithm 1 step 7, tracked_out = base + quantized delta
// (fp32, the representative of the zero bucket, +0, added like any other): inside the coding loop for the chunks
// whose coding never reads base, otherwise chunk by chunk once a chunk's coding no longer needs base.
// tracked_out may be base itself, hence no __restrict__ on the two. Three CTAs per SM instead of four, for the
// registers the rows of base in flight take.
template <bool UPDATE>
__global__ void __launch_bounds__(kEncThreads, UPDATE ? 3 : 4)
encode_kernel(Control* __restrict__ ctl, unsigned long long* __restrict__ tiles, const uint8_t* __restrict__ plane,
              const float* base, const float* __restrict__ cur, uint64_t n, uint8_t* __restrict__ stream,
              float* tracked_out, uint32_t spin_limit, uint32_t ticket_bias, uint32_t two_pass_scan) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ Tables tb;
  __shared__ uint32_t s_chunk_bytes[2][kEncWarps];  // [half][warp]: the pending tile and the one being coded
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_lane_start[2][kEncThreads];  // only for chunks too large for the image area
  __shared__ unsigned long long s_tile_base, s_tile_end;
  __shared__ int s_abort;
  __shared__ uint32_t s_arrived[2];  // warps that have coded their chunk of the tile in this half
  __shared__ uint32_t s_rep[UPDATE ? 256 : 1];  // UPDATE: representative (bit pattern) by plane byte

  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // The table pass may have rejected the vector, or another CTA may already have given up waiting: leave, all
  // threads together (one thread reads the word; a thread-by-thread test could split the CTA if the word changed
  // in between, and the warps that stayed would wait at barriers for the ones that left).
  if (tid == 0) s_abort = ctl->status;
  __syncthreads();
  if (s_abort != 0) return;
  __syncthreads();  // everybody has read s_abort before thread 0 reuses it below
  for (uint32_t b = tid; b < 256; b += kEncThreads) {
    const EncEntry e = ctl->enc[((b & 1u) << 8) | (b >> 1)];
    tb.full[b] = make_uint2(e.code_lo, e.len);
    tb.packed[b] = e.len <= kPackedMaxLen ? (e.len << kPackedLenShift) | e.code_lo : kPackedLong << kPackedLenShift;
    // the table pass has written the stream's symbol table: entry of symbol s at 64 + 16 s, representative at +4
    if (UPDATE) s_rep[b] = *reinterpret_cast<const uint32_t*>(stream + kHeaderBytes + kTableEntryBytes * e.sym + 4);
  }
  __syncthreads();

  const uint32_t nsym = ctl->nsym;
  const bool long_codes = ctl->max_len > 32;
  const KeySource ks{plane, base, cur, ctl->wide != 0};
  const StreamLayout L = stream_layout(n, nsym);
  const uint64_t nchunks = L.nchunks;
  unsigned long long* chunk_index = reinterpret_cast<unsigned long long*>(stream + L.chunk_index_off);
  uint16_t* lane_index = reinterpret_cast<uint16_t*>(stream + L.lane_index_off);
  uint8_t* payload = stream + L.payload_off;
  // how many warps work: as many as can each hold an average chunk (plus 15 %) twice
  const uint64_t avg_bytes = nchunks ? ctl->payload_bits / 8 / nchunks : 0;
  const uint64_t need = avg_bytes + avg_bytes / 7 + 64;
  uint32_t active = kEncWarps;
  while (active > 1 && need > kEncSmem / active / 2) active >>= 1;
  const uint32_t image_words = kEncSmem / active / 8;  // half of the warp's share, in words
  const uint32_t lane_words = image_words / 32;        // rows of the column matrix
  uint32_t* column = s_dyn + (warp % active) * (2 * image_words);  // word k of lane t at column[k*32 + t]
  uint32_t* image = column + image_words;
  const uint32_t packed_addr = smem_addr(tb.packed);

  // Packed table entries of the four plane bytes of `word`.
  auto lookup4 = [&](uint32_t word, uint32_t (&g)[4]) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t b = __byte_perm(word, 0u, 0x4440 + e);  // plane byte of slot e
      // volatile: keeps the loads where they are written, one row ahead of their use
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(g[e]) : "r"(packed_addr + b * 4u));
    }
  };
  // Appends the four codes of `word`, whose packed entries are g. Packed codes have at most 16 bits, so two
  // neighbours are joined into one append of at most 32 bits (half the accumulator and flush work). Only the
  // marker has bit 31 set, so one test per row finds the rare longer codes; that row then appends its four
  // codes one by one from `full`.
  auto put4 = [&](ColumnPacker& pk, uint32_t word, const uint32_t (&g)[4]) {
    if (__any_sync(0xffffffffu, (int)(g[0] | g[1] | g[2] | g[3]) < 0)) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint2 f = tb.full[__byte_perm(word, 0u, 0x4440 + e)];
        pk.put(f.x, f.y);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 4; e += 2) {
        const uint32_t l0 = g[e] >> kPackedLenShift, l1 = g[e + 1] >> kPackedLenShift;
        const uint32_t c0 = g[e] & kPackedCodeMask, c1 = g[e + 1] & kPackedCodeMask;
        pk.put((c0 << l1) | c1, l0 + l1);
      }
    }
  };
  auto fast_chunk = [&](uint64_t cc) { return cc < nchunks && (cc + 1) * kChunkElems <= n && !long_codes && !ks.wide; };

  const uint64_t ntiles = (nchunks + active - 1) / active;

  // The loop is software-pipelined over tiles: a tile's offset is looked up, and its image copied out, only
  // after the *next* tile has been coded. Every earlier tile needs its size before this one can be placed, and
  // with hundreds of tiles in flight some predecessor is always late; looking back right after coding made the
  // whole CTA wait for that straggler for a third of its time. One coding phase later the predecessors' sizes
  // are there. The pending tile lives in the warps' image areas, which coding (phase A) does not touch.
  // What the pending tile needs later is kept in shared memory (its chunk sizes, the lanes' start bits) or
  // recomputed from its number: phase A has no registers to spare.
  bool p_have = false;
  uint32_t p_tile = 0, p_buf = 0;

  if (tid == 0) {
    s_tile = atomicAdd(&ctl->ticket, 1u) + ticket_bias;
    s_abort = 0;
    s_arrived[0] = s_arrived[1] = 0;
  }
  while (true) {
    __syncthreads();  // the ticket taken during the previous iteration is visible; that iteration is done
                      // with the other half of s_chunk_bytes
    const uint64_t tile = s_tile;
    const bool have = tile < ntiles;
    if (!have && !p_have) break;
    const uint32_t buf = p_buf ^ 1u;
    const uint64_t c = tile * active + warp;
    const bool valid = have && warp < active && c < nchunks;
    bool fast = valid && fast_chunk(c);

    // ---- A: code the lane's elements into its column. Lookups run one row (4 elements) ahead of the
    // appends, which depend on each other through the bit accumulator.
    uint32_t lane_bits = 0;
    if (fast) {
      const uint4* ep = reinterpret_cast<const uint4*>(plane + c * kChunkElems) + lane;
      const uint32_t col0 = smem_addr(column) + lane * 4;
      ColumnPacker pk{0u, 0u, 0u, col0, col0 + lane_words * 128};
      uint32_t g0[4], g1[4];
      uint4 cur4 = __ldg(ep);
      lookup4(cur4.x, g0);
      // UPDATE: the tracked state of this chunk is written here, where its plane bytes are in registers; the
      // memory traffic of the update then runs under the coding, which is bound by instruction issue. A chunk on
      // this path never reads base for its coding (not even when it is coded again the slow way), so base may be
      // overwritten at once. Row j of base is requested while row j - 1 is coded.
      const float4* b4 = reinterpret_cast<const float4*>(base + c * kChunkElems) + lane;
      float4* o4 = reinterpret_cast<float4*>(tracked_out + c * kChunkElems) + lane;
      // Rows of base come through a ring of kUpdRows 512-byte slots per warp behind the coding areas, filled by
      // cp.async four rows ahead: that many loads in flight per lane would not fit the registers, and the kernel's
      // L1 is too small to help. A lane reads back only the 16 bytes it copied itself, so no barrier is needed.
      const uint32_t ring = smem_addr(s_dyn) + kEncSmem + warp * (kUpdRows * 512) + lane * 16;
      auto issue_row = [&](int j) {
        if (j < (int)kSteps)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring + (j % kUpdRows) * 512), "l"(b4 + 32 * j)
                       : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");  // also when empty: the wait below counts groups
      };
      if (UPDATE) {
#pragma unroll
        for (int j = 0; j < kUpdRows; ++j) issue_row(j);
      }
      auto update_row = [&](uint32_t word, int j) {
        asm volatile("cp.async.wait_group %0;" ::"n"(kUpdRows - 1) : "memory");  // row j has landed
        float4 b;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w)
                     : "r"(ring + (j % kUpdRows) * 512));
        float4 x;
        x.x = __fadd_rn(b.x, __uint_as_float(s_rep[__byte_perm(word, 0u, 0x4440)]));
        x.y = __fadd_rn(b.y, __uint_as_float(s_rep[__byte_perm(word, 0u, 0x4441)]));
        x.z = __fadd_rn(b.z, __uint_as_float(s_rep[__byte_perm(word, 0u, 0x4442)]));
        x.w = __fadd_rn(b.w, __uint_as_float(s_rep[__byte_perm(word, 0u, 0x4443)]));
        o4[32 * j] = x;
        issue_row(j + kUpdRows);
      };
#pragma unroll 1
      for (int q = 0; q < 8; ++q) {
        const uint4 nxt = __ldg(ep + 32 * (q + 1 < 8 ? q + 1 : q));  // next 16 plane bytes, one step ahead
        lookup4(cur4.y, g1);
        put4(pk, cur4.x, g0);
        if (UPDATE) update_row(cur4.x, 4 * q);
        lookup4(cur4.z, g0);
        put4(pk, cur4.y, g1);
        if (UPDATE) update_row(cur4.y, 4 * q + 1);
        lookup4(cur4.w, g1);
        put4(pk, cur4.z, g0);
        if (UPDATE) update_row(cur4.z, 4 * q + 2);
        lookup4(nxt.x, g0);  // first row of the next step (unused after the last step)
        put4(pk, cur4.w, g1);
        if (UPDATE) update_row(cur4.w, 4 * q + 3);
        cur4 = nxt;
      }
      const bool overflow = pk.nb >= 32 || (pk.nb > 0 && pk.dst >= pk.lim);
      if (__any_sync(0xffffffffu, overflow)) {
        fast = false;  // some lane outgrew its column: redo the chunk the slow way
      } else {
        if (pk.nb > 0) column[((pk.dst - col0) >> 7) * 32 + lane] = pk.lo << (32 - pk.nb);
        lane_bits = ((pk.dst - col0) >> 7) * 32 + pk.nb;
      }
    }
    if (!fast && valid) lane_bits = chunk_slow(ctl->enc, ks, c, lane, n, nullptr, 0);

    // ---- B: lane offsets, lane index, chunk size; the tile's size is published as early as possible
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
    const bool staged = chunk_bytes <= image_words * 4;
    if (!staged) s_lane_start[buf][tid] = lane_start;
    // The warp that gets here first looks up the pending tile's offset (D) while the others are still coding.
    uint32_t arrival = 0;
    if (lane == 0) {
      s_chunk_bytes[buf][warp] = chunk_bytes;
      arrival = atomicAdd(&s_arrived[buf], 1u);
    }
    arrival = __shfl_sync(0xffffffffu, arrival, 0);

    // ---- D: exclusive prefix of the pending tile by decoupled look-back
    if (p_have && arrival == 0) {
      unsigned long long part = 0;  // this lane's share of the sum
      bool abort = false;
      if (two_pass_scan) {
        // the chunk index is already there (encode_scan_kernel): the tile starts where its first chunk starts
        if (lane == 0) part = chunk_index[(uint64_t)p_tile * active];
      } else if (p_tile > 0) {
        long long look = (long long)p_tile - 1;
        uint32_t spins = 0;
        bool done = false;
        while (!done && !abort) {
          // a round reads the kLookBack * 32 descriptors before `look` at once: the nearest tile that
          // already knows its prefix is about one coding phase of tickets back
          unsigned long long st[kLookBack];
#pragma unroll
          for (int u = 0; u < kLookBack; ++u) {
            const long long idx = look - 32 * u - lane;
            st[u] = (kTilePrefix << kTileFlagShift);  // tiles before the first: prefix 0
            if (idx >= 0) st[u] = ld_tile(&tiles[idx]);
          }
          bool retry = false;
#pragma unroll
          for (int u = 0; u < kLookBack; ++u) {
            if (done || abort || retry) continue;
            const uint32_t flag = (uint32_t)(st[u] >> kTileFlagShift);
            const uint32_t m_prefix = __ballot_sync(0xffffffffu, flag == kTilePrefix);
            const uint32_t m_other = __ballot_sync(0xffffffffu, flag != kTilePrefix && flag != kTileAggregate);
            const int first_prefix = m_prefix ? __ffs(m_prefix) - 1 : 32;
            const uint32_t relevant = first_prefix < 32 ? (0xffffffffu >> (31 - first_prefix)) : 0xffffffffu;
            if (m_other & relevant) {
              // a tile without a size yet, or an aborted one
              if (__ballot_sync(0xffffffffu, flag == kTileAbort) & relevant) abort = true;
              else retry = true;  // poll again from `look`, which already skips the complete sub-windows
            } else {
              if ((int)lane <= first_prefix) part += st[u] & kTileValueMask;
              if (first_prefix < 32) done = true;
              else look -= 32;
            }
          }
          if (retry) {
            if (++spins > spin_limit) abort = true;
            else __nanosleep(40);
          }
        }
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
      if (lane == 0) {
        if (abort) {
          set_status(&ctl->status, LC_ERR_TIMEOUT);
          st_tile(&tiles[p_tile], kTileAbort << kTileFlagShift);
          s_abort = 1;
        } else {
          unsigned long long p_tile_bytes = 0;
#pragma unroll
          for (int w = 0; w < (int)kEncWarps; ++w) p_tile_bytes += s_chunk_bytes[p_buf][w];
          if (p_tile > 0 && !two_pass_scan)
            st_tile(&tiles[p_tile], (kTilePrefix << kTileFlagShift) | (part + p_tile_bytes));
          s_abort = 0;
          s_tile_base = part;
          s_tile_end = part + p_tile_bytes;
        }
      }
    }
    __syncthreads();  // all chunk sizes of the new tile, and the pending tile's offset, are known
    if (tid == 0) {
      s_arrived[p_buf] = 0;  // the other half's counter, for the next iteration
      if (have && !two_pass_scan) {
        unsigned long long tile_bytes = 0;
#pragma unroll
        for (int w = 0; w < (int)kEncWarps; ++w) tile_bytes += s_chunk_bytes[buf][w];
        const unsigned long long flag = tile == 0 ? kTilePrefix : kTileAggregate;
        st_tile(&tiles[tile], (flag << kTileFlagShift) | tile_bytes);
      }
    }

    // ---- E: write the pending tile's chunks and their index entries
    if (p_have && !s_abort) {
      unsigned long long chunk_off = s_tile_base;
      for (uint32_t w = 0; w < warp; ++w) chunk_off += s_chunk_bytes[p_buf][w];
      const uint64_t p_c = (uint64_t)p_tile * active + warp;
      const uint32_t p_chunk_bytes = s_chunk_bytes[p_buf][warp];
      const bool p_staged = p_chunk_bytes <= image_words * 4;
      if (warp < active && p_c < nchunks) {
        if (lane == 0) chunk_index[p_c] = chunk_off;
        uint4* dst4 = reinterpret_cast<uint4*>(payload + chunk_off);
        if (p_staged) {
          const uint4* im4 = reinterpret_cast<const uint4*>(image);
          for (uint32_t k = lane; k < p_chunk_bytes / 16; k += 32) dst4[k] = im4[k];
        } else {
          // chunk larger than the image area: OR the bits straight into (zeroed) global memory.
          for (uint32_t k = lane; k < p_chunk_bytes / 16; k += 32) dst4[k] = make_uint4(0, 0, 0, 0);
          __threadfence_block();
          __syncwarp();
          chunk_slow(ctl->enc, ks, p_c, lane, n, reinterpret_cast<uint32_t*>(dst4), s_lane_start[p_buf][tid]);
        }
      }
      if (p_tile == ntiles - 1 && tid == 0) {
        const unsigned long long payload_bytes = s_tile_end;
        chunk_index[nchunks] = payload_bytes;
        *reinterpret_cast<unsigned long long*>(stream + 48) = L.payload_off + payload_bytes;
      }
    }
    // ---- tracked state of the pending tile's chunks (everything that reads base for coding them is done)
    if (UPDATE && p_have && !s_abort) {
      const uint64_t p_c = (uint64_t)p_tile * active + warp;
      if (warp < active && p_c < nchunks && !fast_chunk(p_c)) {  // the others were updated while they were coded
        if ((p_c + 1) * kChunkElems <= n && !ks.wide) {
          const uint4* ep = reinterpret_cast<const uint4*>(plane + p_c * kChunkElems) + lane;
          const float4* b4 = reinterpret_cast<const float4*>(base + p_c * kChunkElems) + lane;
          float4* o4 = reinterpret_cast<float4*>(tracked_out + p_c * kChunkElems) + lane;
#pragma unroll 2
          for (int q = 0; q < 8; ++q) {
            const uint4 w4 = __ldg(ep + 32 * q);  // plane bytes of steps 4q .. 4q+3
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
            float4 b[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) b[r] = b4[32 * (4 * q + r)];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              float4 x;
              x.x = __fadd_rn(b[r].x, __uint_as_float(s_rep[__byte_perm(w[r], 0u, 0x4440)]));
              x.y = __fadd_rn(b[r].y, __uint_as_float(s_rep[__byte_perm(w[r], 0u, 0x4441)]));
              x.z = __fadd_rn(b[r].z, __uint_as_float(s_rep[__byte_perm(w[r], 0u, 0x4442)]));
              x.w = __fadd_rn(b[r].w, __uint_as_float(s_rep[__byte_perm(w[r], 0u, 0x4443)]));
              o4[32 * (4 * q + r)] = x;
            }
          }
        } else {
          // ragged last chunk, or exponents the one-byte plane does not hold: element by element
          for (uint32_t j = 0; j < kSteps; ++j) {
            for (uint32_t e = 0; e < kGroup; ++e) {
              const uint64_t i = p_c * kChunkElems + 128ull * j + 4 * lane + e;
              if (i >= n) continue;
              const uint32_t sym = ctl->enc[ks.key(p_c, j, lane, e)].sym;
              const uint32_t rep = *reinterpret_cast<const uint32_t*>(stream + kHeaderBytes + kTableEntryBytes * sym + 4);
              tracked_out[i] = __fadd_rn(base[i], __uint_as_float(rep));
            }
          }
        }
      }
    }
    if (!have) break;
    // The next ticket is taken now, so that the round trip overlaps the rest of this iteration. (Taking it
    // earlier would only make the tile look late to its successors: its size cannot appear before it is coded.)
    if (tid == 0) s_tile = atomicAdd(&ctl->ticket, 1u) + ticket_bias;
    __syncwarp();  // the warp's image area is free again

    // ---- C: assemble the new tile's chunk image in shared memory
    if (valid && staged) {
      uint4* im4 = reinterpret_cast<uint4*>(image);
      for (uint32_t k = lane; k < chunk_bytes / 16; k += 32) im4[k] = make_uint4(0, 0, 0, 0);
      __syncwarp();
      if (fast) {
        const uint32_t nw = (lane_bits + 31) >> 5, r = lane_start & 31;
        uint32_t* out = image + (lane_start >> 5);
        uint32_t prev = 0;
        for (uint32_t k = 0; k < nw; ++k) {
          const uint32_t w = column[k * 32 + lane];
          atomicOr(out + k, __funnelshift_r(w, prev, r));
          prev = w;
        }
        const uint32_t tail = r ? prev << (32 - r) : 0u;
        if (tail) atomicOr(out + nw, tail);
      } else {
        chunk_slow(ctl->enc, ks, c, lane, n, image, lane_start);
      }
    }
    __syncwarp();
    p_have = true;
    p_tile = (uint32_t)tile;
    p_buf = buf;
  }
}

// ---- two-pass scan: chunk sizes, then their exclusive prefix sum, with no CTA waiting for another ----------

constexpr int kScanThreads = 1024;

// Size in bytes of every chunk (format section 3.3: the chunk's bits rounded up to 16 bytes), one warp per chunk,
// into sizes[c]. Whole chunks whose keys the one-byte plane identifies take their code lengths from a 256-byte
// table in shared memory, 16 plane bytes per load; the vector's partial last chunk and vectors with exponent
// fields >= 128 go through the slow path's counting mode.
__global__ void __launch_bounds__(kEncThreads)
encode_sizes_kernel(const Control* __restrict__ ctl, unsigned long long* __restrict__ sizes,
                    const uint8_t* __restrict__ plane, const float* base, const float* __restrict__ cur, uint64_t n,
                    uint64_t nchunks) {
  __shared__ uint8_t s_len[256];  // code length by plane byte (lengths are at most 63)
  if (ctl->status != 0) return;  // nothing in this kernel writes the word: the same for every thread
  for (uint32_t b = threadIdx.x; b < 256; b += kEncThreads) s_len[b] = (uint8_t)ctl->enc[((b & 1u) << 8) | (b >> 1)].len;
  __syncthreads();
  const uint32_t lane = threadIdx.x & 31;
  const KeySource ks{plane, base, cur, ctl->wide != 0};
  const uint64_t warp0 = (uint64_t)blockIdx.x * kEncWarps + (threadIdx.x >> 5), nwarps = (uint64_t)gridDim.x * kEncWarps;
  for (uint64_t c = warp0; c < nchunks; c += nwarps) {
    uint32_t bits = 0;
    if (!ks.wide && (c + 1) * kChunkElems <= n) {
      const uint4* ep = reinterpret_cast<const uint4*>(plane + c * kChunkElems) + lane;
      uint4 v[kSteps / 4];
#pragma unroll
      for (uint32_t q = 0; q < kSteps / 4; ++q) v[q] = __ldg(ep + 32 * q);
#pragma unroll
      for (uint32_t q = 0; q < kSteps / 4; ++q) {
        const uint32_t w[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
        for (int r = 0; r < 4; ++r)
          bits += s_len[w[r] & 255u] + s_len[(w[r] >> 8) & 255u] + s_len[(w[r] >> 16) & 255u] + s_len[w[r] >> 24];
      }
    } else {
      bits = chunk_slow(ctl->enc, ks, c, lane, n, nullptr, 0);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, d);
    if (lane == 0) sizes[c] = align_up((bits + 7) / 8, kPayloadAlign);
  }
}

// chunk_off[c] = sum of sizes[0..c) for c = 0..nchunks, and the stream's total size into its header. One CTA:
// each thread sums a contiguous run of chunks, the run totals are scanned in shared memory.
__global__ void __launch_bounds__(kScanThreads)
encode_scan_kernel(const Control* __restrict__ ctl, const unsigned long long* __restrict__ sizes, uint64_t n,
                   uint64_t nchunks, uint8_t* __restrict__ stream) {
  __shared__ unsigned long long run_total[kScanThreads];
  if (ctl->status != 0) return;
  const StreamLayout L = stream_layout(n, ctl->nsym);
  unsigned long long* chunk_index = reinterpret_cast<unsigned long long*>(stream + L.chunk_index_off);
  const uint64_t per = (nchunks + kScanThreads - 1) / kScanThreads;
  const uint64_t lo = min(nchunks, per * threadIdx.x), hi = min(nchunks, lo + per);
  unsigned long long sum = 0;
  for (uint64_t c = lo; c < hi; ++c) sum += sizes[c];
  run_total[threadIdx.x] = sum;
  __syncthreads();
  for (int d = 1; d < kScanThreads; d <<= 1) {  // inclusive scan of the run totals
    const unsigned long long v = (int)threadIdx.x >= d ? run_total[threadIdx.x - d] : 0ull;
    __syncthreads();
    run_total[threadIdx.x] += v;
    __syncthreads();
  }
  unsigned long long off = run_total[threadIdx.x] - sum;
  for (uint64_t c = lo; c < hi; ++c) {
    chunk_index[c] = off;
    off += sizes[c];
  }
  if (threadIdx.x == kScanThreads - 1) {
    chunk_index[nchunks] = run_total[kScanThreads - 1];
    *reinterpret_cast<unsigned long long*>(stream + 48) = L.payload_off + run_total[kScanThreads - 1];
  }
}

}  // namespace

cudaError_t launch_encode(Control* ctl, unsigned long long* tiles, const uint8_t* plane, const float* base,
                          const float* cur, uint64_t n, uint8_t* stream, float* tracked_out, const EncodeOptions& opt,
                          cudaStream_t cs) {
  const WorkspaceLayout W = workspace_layout(n);
  if (W.nchunks == 0) return cudaSuccess;
  static int blocks_per_sm[kMaxDevices][2] = {}, sms[kMaxDevices] = {};  // by device ordinal
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  const int v = tracked_out ? 1 : 0;
  if (blocks_per_sm[dev][v] == 0) {
    const void* fn = v ? reinterpret_cast<const void*>(encode_kernel<true>) : reinterpret_cast<const void*>(encode_kernel<false>);
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kEncSmem + (v ? kUpdSmem : 0));
    if (e != cudaSuccess) return e;
    int nsm = 0;
    if ((e = cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    int bps = 0;
    e = v ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, encode_kernel<true>, kEncThreads, kEncSmem + kUpdSmem)
          : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, encode_kernel<false>, kEncThreads, kEncSmem);
    if (e != cudaSuccess) return e;
    sms[dev] = nsm;
    blocks_per_sm[dev][v] = bps > 0 ? bps : 1;
  }
  const uint64_t want = (W.nchunks + kEncWarps - 1) / kEncWarps;
  const uint64_t full = (uint64_t)sms[dev] * blocks_per_sm[dev][v];
  const unsigned grid = (unsigned)(want < full ? want : full);
  if (opt.two_pass_scan) {
    // tiles[] (zeroed by the caller, one entry per chunk) holds the chunk sizes in this mode
    encode_sizes_kernel<<<grid, kEncThreads, 0, cs>>>(ctl, tiles, plane, base, cur, n, W.nchunks);
    encode_scan_kernel<<<1, kScanThreads, 0, cs>>>(ctl, tiles, n, W.nchunks, stream);
    if (cudaGetLastError() != cudaSuccess) return cudaErrorLaunchFailure;
  }
  const uint32_t two = opt.two_pass_scan ? 1u : 0u;
  if (v)
    encode_kernel<true><<<grid, kEncThreads, kEncSmem + kUpdSmem, cs>>>(ctl, tiles, plane, base, cur, n, stream, tracked_out,
                                                                       opt.spin_limit, opt.ticket_bias, two);
  else
    encode_kernel<false><<<grid, kEncThreads, kEncSmem, cs>>>(ctl, tiles, plane, base, cur, n, stream, nullptr,
                                                              opt.spin_limit, opt.ticket_bias, two);
  return cudaGetLastError();
}

}  // namespace lc
