// The table pass as a function of one CTA of kTableThreads threads (Section 3.1.1: priority promotion and
// representatives; Section 3.1.2: Huffman code; format sections 1.2-1.8): shared by table_kernel and by the
// single-CTA kernel for small vectors. Returns false (for every thread alike) if it left no table behind: an earlier
// pass had failed, or the vector is not encodable.
#pragma once
#include "lc_common.cuh"

namespace lc {

constexpr int kTableThreads = 512;
constexpr int kMaxSym = kMaxSymbols;

__device__ __forceinline__ void store_le(uint8_t* p, uint64_t v, int bytes) {
  for (int b = 0; b < bytes; ++b) p[b] = (uint8_t)(v >> (8 * b));
}

__device__ __forceinline__ bool table_pass(Control* __restrict__ ctl, uint64_t n, int nbits, uint8_t* __restrict__ stream,
                                           int wide_ok, int fixed, const ShardStats* __restrict__ whole,
                                           uint8_t* __restrict__ cache, int mean) {
  __shared__ uint32_t warp_cand[16];
  __shared__ uint16_t sym_of_key[kKeys];
  __shared__ unsigned long long sym_count[kMaxSym];
  __shared__ uint32_t sym_key[kMaxSym];
  __shared__ uint32_t sym_rep[kMaxSym];
  __shared__ uint32_t sym_len[kMaxSym];
  __shared__ unsigned long long sym_code[kMaxSym];
  __shared__ unsigned long long node_w[2 * kMaxSym];
  __shared__ uint16_t node_parent[2 * kMaxSym];
  __shared__ uint16_t node_depth[2 * kMaxSym];
  __shared__ uint16_t leaf_sym[kMaxSym];
  __shared__ uint16_t canon_order[kMaxSym];
  __shared__ uint32_t s_maxlen;
  __shared__ unsigned long long s_kept_total, s_payload_bits;
  __shared__ unsigned long long s_cached_bits;  // payload size with the lengths of the cache row

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  // The statistics that decide the table: this vector's own, or those of the whole vector it is a shard of.
  const unsigned long long* g_count = whole ? whole->count : ctl->count;
  const uint32_t* g_inv_min = whole ? whole->inv_min : ctl->inv_min;
  const uint32_t* g_max_bits = whole ? whole->max_bits : ctl->max_bits;
  __shared__ unsigned long long s_whole_total;
  __shared__ unsigned long long sym_local[kMaxSym];  // the table's counts: this vector's own elements per symbol

  // ---- an earlier pass of the same call has failed (lc_merge: a stream was rejected): leave no stream behind
  if (ctl->status != 0) {  // nothing in this kernel has written the word yet: the same for every thread
    if (tid < 64) stream[tid] = 0;
    return false;
  }

  // ---- non-finite deltas make the vector unencodable ------------------------------------------
  const bool bad = (tid == 255 || tid == 511) && g_count[tid] != 0;
  if (__syncthreads_or(bad)) {
    if (tid == 0) {
      set_status(&ctl->status, LC_ERR_NONFINITE);
      for (int b = 0; b < 64; ++b) stream[b] = 0;
    }
    return false;
  }

  // ---- does the one-byte key plane identify every bucket? (only if all exponent fields are < 128)
  const bool big = (tid & 255) >= 128 && (g_count[tid] != 0 || ctl->count[tid] != 0);
  const int wide = __syncthreads_or(big);
  if (wide && !wide_ok) {
    // the caller has released base and cur, and the one-byte keys do not identify the buckets of this vector
    if (tid == 0) {
      set_status(&ctl->status, LC_ERR_RANGE);
      for (int b = 0; b < 64; ++b) stream[b] = 0;
    }
    return false;
  }

  // ---- priority promotion -------------------------------------------------------------------------
  // thread `tid` < 508 looks at the key of priority position tid: exponent descending, + before -.
  uint32_t key = 0;
  unsigned long long cnt = 0;
  bool cand = false;
  if (tid < 508) {
    const uint32_t E = 254 - (tid >> 1), s = tid & 1;
    key = 256 * s + E;
    cnt = g_count[key];
    cand = cnt != 0;
  }
  if (tid < kMaxSym) {
    sym_count[tid] = 0;
    sym_len[tid] = 0;
    sym_code[tid] = 0;
    sym_key[tid] = 0;
    sym_rep[tid] = 0;
  }
  sym_of_key[tid] = 0;
  if (tid == 0) {
    s_kept_total = 0;
    s_payload_bits = 0;
    s_maxlen = 0;
    s_whole_total = 0;
    s_cached_bits = 0;
  }
  sym_local[tid] = 0;
  const uint32_t ballot = __ballot_sync(0xffffffffu, cand);
  if (lane == 0) warp_cand[warp] = __popc(ballot);
  __syncthreads();
  uint32_t rank = __popc(ballot & ((1u << lane) - 1));
  uint32_t ncand = 0;
  for (int w = 0; w < 16; ++w) {
    if (w < warp) rank += warp_cand[w];
    ncand += warp_cand[w];
  }
  const uint32_t keep = min((1u << nbits) - 1u, ncand);
  const uint32_t nsym = keep + 1;
  if (cand && rank < keep) {
    const uint32_t sym = rank + 1;
    sym_of_key[key] = (uint16_t)sym;
    sym_count[sym] = cnt;
    sym_key[sym] = key;
    // midrange of two values with the same sign and exponent, rounded to nearest even, on mantissas.
    sym_local[sym] = ctl->count[key];
    const uint32_t mmin = (~g_inv_min[key]) & 0x7FFFFFu;
    const uint32_t mmax = g_max_bits[key] & 0x7FFFFFu;
    const uint32_t t = mmin + mmax;
    uint32_t mr = t >> 1;
    if ((t & 1u) && (mr & 1u)) mr += 1;
    if (mean) {
      // variant (format section 1.8): mean of the mantissa fields, rounded to nearest, ties to even; it cannot reach
      // 2^23 because it does not exceed the largest field
      const unsigned long long sum = ctl->mant_sum[key];
      unsigned long long q = sum / cnt;
      const unsigned long long r = sum - q * cnt;
      if (2 * r > cnt || (2 * r == cnt && (q & 1ull))) q += 1;
      mr = (uint32_t)q;
    }
    sym_rep[sym] = (key << 23) | mr;
    atomicAdd(&s_kept_total, cnt);
  }
  if (whole) atomicAdd(&s_whole_total, g_count[tid]);  // elements of the whole vector
  __syncthreads();
  if (tid == 0) {
    sym_count[0] = (whole ? s_whole_total : n) - s_kept_total;
    unsigned long long kept_local = 0;
    for (uint32_t j = 1; j < nsym; ++j) kept_local += sym_local[j];
    sym_local[0] = n - kept_local;
  }
  __syncthreads();

  // ---- Huffman lengths: two-queue construction ----------------------------------------------------
  // queue A = used symbols sorted by (count, id), found with a rank sort.
  bool used = false;
  unsigned long long my_count = 0;
  if (tid < (int)nsym) {
    my_count = sym_count[tid];
    used = my_count != 0;
  }
  const uint32_t used_ballot = __ballot_sync(0xffffffffu, used);
  if (lane == 0) warp_cand[warp] = __popc(used_ballot);
  __syncthreads();
  uint32_t nused = 0;
  for (int w = 0; w < 16; ++w) nused += warp_cand[w];
  if (fixed) {
    // fixed-width codes (format section 1.5): every symbol, used or not, takes ceil(log2 nsym) bits; its code is its id
    uint32_t width = 0;
    while ((1u << width) < nsym) width += 1;
    if (tid < (int)nsym) {
      sym_len[tid] = width;
      sym_code[tid] = (unsigned long long)tid;
    }
    if (tid == 0) {
      s_maxlen = width;
      s_payload_bits = n * width;
    }
  }
  // ---- code-table caching (Section 3.2; format section 1.7): a valid row for this number of used symbols gives
  // the r-th most frequent symbol its r-th length, if the payload then stays within n * nbits bits
  uint8_t* row = (cache && !fixed && nused >= 2) ? cache + (size_t)kLengthCacheRow * (nused - 1) : nullptr;
  uint32_t offered = 0;
  if (row && row[0] != 0 && used) {  // row[0] is read before anything in this kernel writes the row
    uint32_t r = 0;
    for (uint32_t j = 0; j < nsym; ++j) {
      const unsigned long long cj = sym_count[j];
      if (cj != 0 && (cj > my_count || (cj == my_count && (int)j < tid))) r += 1;
    }
    offered = row[r];
    atomicAdd(&s_cached_bits, my_count * offered);
  }
  const bool row_valid = row && row[0] != 0;
  __syncthreads();
  const bool hit = row_valid && s_cached_bits <= n * (unsigned long long)nbits;
  if (hit) {
    if (used) {
      sym_len[tid] = offered;
      atomicMax(&s_maxlen, offered);
    }
  }
  if (used && !fixed && !hit) {
    uint32_t r = 0;
    for (uint32_t j = 0; j < nsym; ++j) {
      const unsigned long long cj = sym_count[j];
      if (cj != 0 && (cj < my_count || (cj == my_count && (int)j < tid))) r += 1;
    }
    node_w[r] = my_count;
    leaf_sym[r] = (uint16_t)tid;
  }
  __syncthreads();
  if (tid == 0 && nused >= 2 && !fixed && !hit) {
    uint32_t front_a = 0, front_b = nused, next = nused;
    for (uint32_t merge = 0; merge + 1 < nused; ++merge) {
      uint32_t pick[2];
      for (int q = 0; q < 2; ++q) {
        const bool a_has = front_a < nused, b_has = front_b < next;
        if (a_has && (!b_has || node_w[front_a] <= node_w[front_b])) pick[q] = front_a++;
        else pick[q] = front_b++;
      }
      node_w[next] = node_w[pick[0]] + node_w[pick[1]];
      node_parent[pick[0]] = (uint16_t)next;
      node_parent[pick[1]] = (uint16_t)next;
      next += 1;
    }
    // depths, from the root (the last node) down; parents always have larger indices.
    const uint32_t root = next - 1;
    node_depth[root] = 0;
    for (int v = (int)root - 1; v >= 0; --v) node_depth[v] = node_depth[node_parent[v]] + 1;
    uint32_t maxlen = 0;
    unsigned long long bits = 0;
    for (uint32_t r = 0; r < nused; ++r) {
      sym_len[leaf_sym[r]] = node_depth[r];
      maxlen = max(maxlen, (uint32_t)node_depth[r]);
      bits += node_w[r] * node_depth[r];
    }
    s_maxlen = maxlen;
    s_payload_bits = bits;
  }
  __syncthreads();

  // ---- canonical codes: used symbols sorted by (len, id) -------------------------------------------
  if (used && nused >= 2 && !fixed) {
    const uint32_t my_len = sym_len[tid];
    uint32_t r = 0;
    for (uint32_t j = 0; j < nsym; ++j) {
      const uint32_t lj = sym_len[j];
      if (lj != 0 && (lj < my_len || (lj == my_len && (int)j < tid))) r += 1;
    }
    canon_order[r] = (uint16_t)tid;
    if (row && !hit) row[r] = (uint8_t)my_len;  // a miss stores the new lengths, ascending
  }
  if (row && !hit && tid >= (int)nused) row[tid] = 0;
  __syncthreads();
  if (tid == 0 && nused >= 2 && !fixed) {
    unsigned long long code = 0;
    uint32_t prev_len = 0;
    for (uint32_t r = 0; r < nused; ++r) {
      const uint32_t j = canon_order[r];
      if (r > 0) code = (code + 1) << (sym_len[j] - prev_len);
      sym_code[j] = code;
      prev_len = sym_len[j];
    }
  }
  __syncthreads();

  // ---- payload size: this vector's own elements, with the lengths just found --------------------------
  if (tid == 0) s_payload_bits = 0;
  __syncthreads();
  if (tid < (int)nsym) atomicAdd(&s_payload_bits, sym_local[tid] * sym_len[tid]);
  __syncthreads();

  // ---- outputs ---------------------------------------------------------------------------------------
  {
    const uint32_t sym = sym_of_key[tid];
    EncEntry e;
    e.code_lo = (uint32_t)sym_code[sym];
    e.code_hi = (uint32_t)(sym_code[sym] >> 32);
    e.len = sym_len[sym];
    e.sym = sym;
    ctl->enc[tid] = e;
  }
  const StreamLayout L = stream_layout(n, nsym);
  if (tid < (int)nsym) {
    uint8_t* e = stream + L.table_off + 16 * tid;
    store_le(e, sym_key[tid], 2);
    e[2] = (uint8_t)sym_len[tid];
    e[3] = 0;
    store_le(e + 4, sym_rep[tid], 4);
    store_le(e + 8, sym_local[tid], 8);
  }
  if (tid == 0) {
    ctl->nsym = nsym;
    ctl->wide = wide ? 1u : 0u;
    ctl->max_len = s_maxlen;
    ctl->payload_bits = s_payload_bits;
    uint8_t* h = stream;
    h[0] = 'L'; h[1] = 'C'; h[2] = 'C'; h[3] = '1';
    store_le(h + 4, 1, 2);
    h[6] = (uint8_t)nbits;
    h[7] = (uint8_t)((fixed ? 1 : 0) | (whole ? 2 : 0) | (hit ? 4 : 0) | (mean ? 8 : 0));
    store_le(h + 8, n, 8);
    store_le(h + 16, nsym, 4);
    store_le(h + 20, s_maxlen, 4);
    store_le(h + 24, kChunkElems, 4);
    store_le(h + 28, kLanes, 2);
    store_le(h + 30, kGroup, 2);
    store_le(h + 32, L.nchunks, 4);
    store_le(h + 36, kPayloadAlign, 4);
    store_le(h + 40, s_payload_bits, 8);
    store_le(h + 56, L.payload_off, 8);
    // bytes between the lane index and the payload are zero.
    for (uint64_t p = L.lane_index_off + 64 * L.nchunks; p < L.payload_off; ++p) stream[p] = 0;
    if (L.nchunks == 0) {
      // nothing for the encode pass to do: finish the stream here.
      store_le(stream + L.chunk_index_off, 0, 8);
      store_le(h + 48, L.payload_off, 8);
    }
  }
  return true;
}

}  // namespace lc
