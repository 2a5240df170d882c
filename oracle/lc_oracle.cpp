// CPU oracle for the LC-Checkpoint compress and recovery passes.
//
// TEST INFRASTRUCTURE ONLY. This file is the plain, slow, single-threaded statement of what the
// method computes, written step by step from the paper (arxiv 2009.13003) and from the stream
// format text in docs/FORMAT.md. It exists to check the CUDA library and to serve as the timed CPU
// baseline. Only the tests, the smoke check and the benchmark's CPU-baseline leg may load it; the
// product never does. It shares no code with the CUDA path.
//
// Everything is done the obvious way: one loop per step, bits written one at a time, decoding by
// walking an explicit code tree one bit at a time.
//
// Pins (see tests/test_oracle_*.py): hand-worked vectors with known bit patterns, byte-exact golden
// streams written by hand from the format text, brute-force optimal prefix codes on tiny alphabets,
// Kraft equality, entropy bound, textbook code-length cases, the integer midrange identity, the
// paper's worked size example (Section 3.1.1: n=10, k=5 -> 190 bits, rate 1.68), round trips and the
// chain identity of Algorithm 1. The helpers are pinned to the main functions: lco_apply_quantized to
// lco_recover of lco_compress, lco_compress_chunks to slices of lco_compress's stream, the threaded
// timing mode to the single-threaded bytes, lco_merge to the idempotence of quantization over a zero
// base (the merged stream of one stream is that stream) and to Algorithm 1 step 7 applied to the
// recovered state. The length cache of Section 3.2 (lco_cached_lengths, lco_compress_cached) is pinned by hand-worked
// rows and assignments, by byte equality with the plain stream on an empty cache, and by a cached stream
// recovering the plain stream's state with more payload bits than the plain stream's optimal code. The mean
// variant (lco_bucket_mean, lco_compress_mean) is pinned by hand-worked buckets (ties, thirds of an ulp, both ends
// of the exponent range) and by exact rational arithmetic on random buckets and on the buckets of a stream.
// Parity unpinned: the whole-pipeline result on the paper's own training deltas (its figures carry
// the only values and they are not available); only the loose size ranges of Section 4.3 apply.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

constexpr int LCO_OK = 0;
constexpr int LCO_ERR_ARG = -1;
constexpr int LCO_ERR_CAPACITY = -2;
constexpr int LCO_ERR_NONFINITE = -3;
constexpr int LCO_ERR_FORMAT = -4;
constexpr int LCO_ERR_MISMATCH = -5;

constexpr uint64_t kChunkElems = 4096;  // elements per chunk (format section 2)
constexpr uint64_t kLanes = 32;         // lane sub-streams per chunk
constexpr uint64_t kGroup = 4;          // consecutive elements a lane takes per step
constexpr uint64_t kSteps = kChunkElems / (kLanes * kGroup);

typedef uint16_t sym_t;  // symbol ids reach 508 when every bucket is kept (nbits = 9)

uint32_t float_bits(float f) {
  uint32_t u;
  std::memcpy(&u, &f, sizeof u);
  return u;
}

float bits_float(uint32_t u) {
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

uint64_t align16(uint64_t x) { return (x + 15) / 16 * 16; }

// Section 3.1.1, exponent-based quantization: the bucket of a value is (sign, exponent field).
int bucket_key(float d) {
  const uint32_t u = float_bits(d);
  const int s = static_cast<int>(u >> 31);
  const int E = static_cast<int>((u >> 23) & 255u);
  return 256 * s + E;
}

struct Bucket {
  uint64_t count = 0;
  float vmin = 0.0f;  // smallest value seen in the bucket
  float vmax = 0.0f;  // largest value seen in the bucket
  unsigned __int128 sig_sum = 0;  // sum of the 24-bit integer significands of the bucket's values (mean variant)
};

// Algorithm 1 step 4 (delta against the tracked state) followed by the bucketing of Section 3.1.1.
void delta_buckets(const float* base, const float* cur, uint64_t n, Bucket* buckets /*[512]*/) {
  for (int k = 0; k < 512; ++k) buckets[k] = Bucket();
  for (uint64_t i = 0; i < n; ++i) {
    const float d = cur[i] - base[i];
    Bucket& b = buckets[bucket_key(d)];
    if (b.count == 0) {
      b.vmin = d;
      b.vmax = d;
    } else {
      if (d < b.vmin) b.vmin = d;
      if (d > b.vmax) b.vmax = d;
    }
    b.count += 1;
    b.sig_sum += (float_bits(d) & 0x7FFFFFu) | 0x800000u;
  }
}

// Variant (format section 1.8): the bucket is represented by the MEAN of its values instead of the average of its
// maximum and minimum. Every value of a bucket is sign * 2^(E-150) * (its 24-bit integer significand), so the exact
// mean is that scale times the mean of the integers; rounding the latter to the nearest integer, ties to even,
// rounds the exact mean to fp32 (the mean lies in the bucket's binade, where fp32 values are those integers).
float bucket_mean(int key, unsigned __int128 sig_sum, uint64_t count) {
  const unsigned __int128 q = sig_sum / count, r = sig_sum % count;
  uint64_t sig = static_cast<uint64_t>(q);
  if (2 * r > count || (2 * r == count && (sig & 1u))) sig += 1;
  const double magnitude = std::ldexp(static_cast<double>(sig), (key & 255) - 150);
  return static_cast<float>((key >> 8) ? -magnitude : magnitude);
}

struct Selection {
  int nsym = 1;                 // K + 1
  int key_of_symbol[512] = {};  // key_of_symbol[0] is 0 by convention
  int symbol_of_key[512] = {};  // 0 for everything that is not kept
};

// Section 3.1.1, priority promotion: keep the 2^x - 1 occupied buckets with the largest exponent
// (positive before negative at equal exponent); everything else falls into the zero bucket.
Selection priority_promotion(const Bucket* buckets, int nbits) {
  Selection sel;
  const int keep_max = (1 << nbits) - 1;
  int kept = 0;
  for (int E = 254; E >= 1; --E) {
    for (int s = 0; s <= 1; ++s) {
      const int key = 256 * s + E;
      if (buckets[key].count > 0 && kept < keep_max) {
        kept += 1;
        sel.key_of_symbol[kept] = key;
        sel.symbol_of_key[key] = kept;
      }
    }
  }
  sel.nsym = kept + 1;
  return sel;
}

// Section 3.1.1: a bucket is represented by the average of its maximum and minimum values. The sum
// of two floats and its half are exact in double, so the only rounding is the final one to fp32.
float midrange(float vmin, float vmax) {
  const double mid = (static_cast<double>(vmin) + static_cast<double>(vmax)) * 0.5;
  return static_cast<float>(mid);
}

// Section 3.1.2: Huffman code lengths by the two-queue construction, ties resolved as the format
// text says (leaves ordered by count then id; a leaf wins over an internal node of equal weight).
void huffman_lengths(const uint64_t* count, int nsym, int* len /*[nsym]*/) {
  for (int j = 0; j < nsym; ++j) len[j] = 0;
  std::vector<int> used;
  for (int j = 0; j < nsym; ++j)
    if (count[j] > 0) used.push_back(j);
  if (used.size() < 2) return;

  std::stable_sort(used.begin(), used.end(), [&](int a, int b) {
    if (count[a] != count[b]) return count[a] < count[b];
    return a < b;
  });

  struct Node {
    uint64_t weight;
    int parent;
  };
  std::vector<Node> nodes;  // first the leaves in queue-A order, then internal nodes in creation order
  for (int j : used) nodes.push_back(Node{count[j], -1});
  const size_t nleaves = used.size();
  size_t front_a = 0;        // next unmerged leaf
  size_t front_b = nleaves;  // next unmerged internal node

  auto take_smallest = [&]() -> size_t {
    const bool a_has = front_a < nleaves;
    const bool b_has = front_b < nodes.size();
    if (a_has && (!b_has || nodes[front_a].weight <= nodes[front_b].weight)) return front_a++;
    return front_b++;
  };

  for (size_t merge = 0; merge + 1 < nleaves; ++merge) {
    const size_t x = take_smallest();
    const size_t y = take_smallest();
    const int parent = static_cast<int>(nodes.size());
    nodes.push_back(Node{nodes[x].weight + nodes[y].weight, -1});
    nodes[x].parent = parent;
    nodes[y].parent = parent;
  }

  for (size_t leaf = 0; leaf < nleaves; ++leaf) {
    int depth = 0;
    for (int v = static_cast<int>(leaf); nodes[v].parent >= 0; v = nodes[v].parent) depth += 1;
    len[used[leaf]] = depth;
  }
}

// Canonical code assignment (format section 1.4).
void canonical_codes(const int* len, int nsym, uint64_t* code /*[nsym]*/) {
  std::vector<int> order;
  for (int j = 0; j < nsym; ++j) {
    code[j] = 0;
    if (len[j] > 0) order.push_back(j);
  }
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    if (len[a] != len[b]) return len[a] < len[b];
    return a < b;
  });
  uint64_t next = 0;
  int prev_len = 0;
  for (size_t r = 0; r < order.size(); ++r) {
    const int j = order[r];
    if (r > 0) next = (next + 1) << (len[j] - prev_len);
    code[j] = next;
    prev_len = len[j];
  }
}

struct Table {
  int nbits = 0;
  int nsym = 1;
  int max_len = 0;
  int fixed = 0;   // 1: fixed-width codes (format section 1.5) instead of the Huffman code
  int shared = 0;  // 1: the table was built from a larger vector than the stream codes (format section 1.6)
  int cached = 0;  // 1: the code lengths were taken from a length cache (format section 1.7)
  int mean = 0;    // 1: representatives are bucket means (format section 1.8)
  int key[512] = {};
  int len[512] = {};
  float rep[512] = {};
  uint64_t count[512] = {};
  uint64_t code[512] = {};
};

// Steps of Sections 3.1.1-3.1.2 that turn bucket statistics into the symbol table.
// Section 3.2, "Huffman Code Table Caching": the code table of an earlier snapshot with the same number of buckets
// is used again, the buckets only being sorted by their numbers of entries. The cache (format section 1.7) has one
// row of 512 bytes per number u of used symbols, row u - 1: the u code lengths in ascending order, valid if its
// first byte is not 0. A valid row gives the r-th most frequent used symbol (ties: smaller id first) the r-th
// length, provided the payload then stays within n * nbits bits (the stream bound); otherwise the Huffman lengths
// are built and written to the row. Returns 1 if the lengths came from the cache.
constexpr int kCacheRowBytes = 512;
int cached_lengths(const uint64_t* count, int nsym, int nbits, uint64_t n, uint8_t* cache, int* len /*[nsym]*/) {
  std::vector<int> used;
  for (int j = 0; j < nsym; ++j)
    if (count[j] > 0) used.push_back(j);
  const int u = static_cast<int>(used.size());
  if (u < 2) {
    for (int j = 0; j < nsym; ++j) len[j] = 0;
    return 0;
  }
  uint8_t* row = cache + static_cast<size_t>(kCacheRowBytes) * (u - 1);
  if (row[0] != 0) {
    std::stable_sort(used.begin(), used.end(), [&](int a, int b) {
      if (count[a] != count[b]) return count[a] > count[b];
      return a < b;
    });
    unsigned __int128 bits = 0;
    for (int r = 0; r < u; ++r) bits += static_cast<unsigned __int128>(count[used[r]]) * row[r];
    if (bits <= static_cast<unsigned __int128>(n) * static_cast<unsigned>(nbits)) {
      for (int j = 0; j < nsym; ++j) len[j] = 0;
      for (int r = 0; r < u; ++r) len[used[r]] = row[r];
      return 1;
    }
  }
  huffman_lengths(count, nsym, len);
  std::vector<int> sorted;
  for (int j = 0; j < nsym; ++j)
    if (count[j] > 0) sorted.push_back(len[j]);
  std::sort(sorted.begin(), sorted.end());
  for (int r = 0; r < kCacheRowBytes; ++r) row[r] = r < u ? static_cast<uint8_t>(sorted[r]) : 0;
  return 0;
}

int build_table(const Bucket* buckets, uint64_t n, int nbits, Table* t, Selection* sel_out, int fixed = 0,
                uint8_t* cache = nullptr, int mean = 0) {
  for (int s = 0; s <= 1; ++s)
    if (buckets[256 * s + 255].count > 0) return LCO_ERR_NONFINITE;
  const Selection sel = priority_promotion(buckets, nbits);
  *t = Table();
  t->nbits = nbits;
  t->nsym = sel.nsym;
  uint64_t kept_total = 0;
  for (int j = 1; j < sel.nsym; ++j) {
    const Bucket& b = buckets[sel.key_of_symbol[j]];
    t->key[j] = sel.key_of_symbol[j];
    t->rep[j] = mean ? bucket_mean(sel.key_of_symbol[j], b.sig_sum, b.count) : midrange(b.vmin, b.vmax);
    t->count[j] = b.count;
    kept_total += b.count;
  }
  t->key[0] = 0;
  t->rep[0] = 0.0f;
  t->count[0] = n - kept_total;
  t->fixed = fixed;
  t->mean = mean;
  if (fixed) {
    // Section 3.1.1's size model: every bucket index takes ceil(log2 k) bits; the code of a symbol is its id.
    int width = 0;
    while ((1 << width) < t->nsym) width += 1;
    for (int j = 0; j < t->nsym; ++j) {
      t->len[j] = width;
      t->code[j] = static_cast<uint64_t>(j);
    }
  } else {
    if (cache) t->cached = cached_lengths(t->count, t->nsym, nbits, n, cache, t->len);
    else huffman_lengths(t->count, t->nsym, t->len);
    canonical_codes(t->len, t->nsym, t->code);
  }
  for (int j = 0; j < t->nsym; ++j) t->max_len = std::max(t->max_len, t->len[j]);
  if (sel_out) *sel_out = sel;
  return LCO_OK;
}

// Little-endian field writers / readers.
void put_le(uint8_t* p, uint64_t v, int bytes) {
  for (int b = 0; b < bytes; ++b) p[b] = static_cast<uint8_t>(v >> (8 * b));
}
uint64_t get_le(const uint8_t* p, int bytes) {
  uint64_t v = 0;
  for (int b = 0; b < bytes; ++b) v |= static_cast<uint64_t>(p[b]) << (8 * b);
  return v;
}

// Sets bit `b` of a chunk (format section 2: word b>>5, bit position 31-(b&31), little-endian words).
void set_chunk_bit(uint8_t* chunk, uint64_t b) {
  const uint64_t word = b >> 5;
  const int pos = 31 - static_cast<int>(b & 31);
  chunk[4 * word + pos / 8] |= static_cast<uint8_t>(1u << (pos % 8));
}
int get_chunk_bit(const uint8_t* chunk, uint64_t b) {
  const uint64_t word = b >> 5;
  const int pos = 31 - static_cast<int>(b & 31);
  return (chunk[4 * word + pos / 8] >> (pos % 8)) & 1;
}

struct Layout {
  uint64_t nchunks, table_off, chunk_index_off, lane_index_off, payload_off;
};

Layout layout_for(uint64_t n, int nsym) {
  Layout L;
  L.nchunks = (n + kChunkElems - 1) / kChunkElems;
  L.table_off = 64;
  L.chunk_index_off = L.table_off + 16ull * nsym;
  L.lane_index_off = L.chunk_index_off + 8 * (L.nchunks + 1);
  L.payload_off = align16(L.lane_index_off + 64 * L.nchunks);
  return L;
}

uint64_t stream_bound(uint64_t n, int nbits) {
  const Layout L = layout_for(n, 1 << nbits);
  return L.payload_off + (n * static_cast<uint64_t>(nbits) + 7) / 8 + 16 * L.nchunks;
}

// The element a lane codes at (step j, slot e) of chunk c (format section 2).
uint64_t element_index(uint64_t c, uint64_t lane, uint64_t j, uint64_t e) {
  return kChunkElems * c + kLanes * kGroup * j + kGroup * lane + e;
}

// Codes one chunk (format section 2): writes the 32 lane bit counts (u16 each) and the chunk's bytes,
// returns the chunk's size in bytes (a multiple of 16).
uint64_t encode_chunk(const float* base, const float* cur, uint64_t n, const Table& t, const Selection& sel,
                      uint64_t c, uint8_t* lane_index /*[64]*/, uint8_t* chunk, uint64_t* chunk_bits_out) {
  // first the lane lengths, to know the chunk size, then the bits.
  uint64_t chunk_bits = 0;
  for (uint64_t lane = 0; lane < kLanes; ++lane) {
    uint64_t lane_bits = 0;
    for (uint64_t j = 0; j < kSteps; ++j)
      for (uint64_t e = 0; e < kGroup; ++e) {
        const uint64_t i = element_index(c, lane, j, e);
        if (i < n) lane_bits += t.len[sel.symbol_of_key[bucket_key(cur[i] - base[i])]];
      }
    put_le(lane_index + 2 * lane, lane_bits, 2);
    chunk_bits += lane_bits;
  }
  const uint64_t chunk_bytes = align16((chunk_bits + 7) / 8);
  std::memset(chunk, 0, chunk_bytes);
  uint64_t bit = 0;
  for (uint64_t lane = 0; lane < kLanes; ++lane)
    for (uint64_t j = 0; j < kSteps; ++j)
      for (uint64_t e = 0; e < kGroup; ++e) {
        const uint64_t i = element_index(c, lane, j, e);
        if (i >= n) continue;
        const int symbol = sel.symbol_of_key[bucket_key(cur[i] - base[i])];
        for (int b = t.len[symbol] - 1; b >= 0; --b) {
          if ((t.code[symbol] >> b) & 1) set_chunk_bit(chunk, bit);
          bit += 1;
        }
      }
  *chunk_bits_out = chunk_bits;
  return chunk_bytes;
}

struct Parsed {
  Table table;
  uint64_t n = 0;
  Layout layout{};
  uint64_t payload_bits = 0;
  uint64_t total_bytes = 0;
};

// Reads and validates header + table (format sections 3 and 4).
int parse_stream(const uint8_t* s, uint64_t bytes, Parsed* out) {
  if (bytes < 64) return LCO_ERR_FORMAT;
  if (!(s[0] == 'L' && s[1] == 'C' && s[2] == 'C' && s[3] == '1')) return LCO_ERR_FORMAT;
  if (get_le(s + 4, 2) != 1) return LCO_ERR_FORMAT;
  const int nbits = static_cast<int>(s[6]);
  if (nbits < 1 || nbits > 9 || s[7] > 15) return LCO_ERR_FORMAT;
  const int fixed = static_cast<int>(s[7] & 1), shared = static_cast<int>((s[7] >> 1) & 1);
  const int cached = static_cast<int>((s[7] >> 2) & 1), mean = static_cast<int>((s[7] >> 3) & 1);
  if ((cached || mean) && (s[7] & (s[7] - 1)) != 0) return LCO_ERR_FORMAT;  // bits 2 and 3 each go alone
  const uint64_t n = get_le(s + 8, 8);
  const uint64_t nsym = get_le(s + 16, 4);
  const uint64_t max_len = get_le(s + 20, 4);
  if (n >= (1ull << 32)) return LCO_ERR_FORMAT;
  if (nsym < 1 || nsym > (1ull << nbits)) return LCO_ERR_FORMAT;
  if (get_le(s + 24, 4) != kChunkElems || get_le(s + 28, 2) != kLanes || get_le(s + 30, 2) != kGroup)
    return LCO_ERR_FORMAT;
  const Layout L = layout_for(n, static_cast<int>(nsym));
  if (get_le(s + 32, 4) != L.nchunks || get_le(s + 36, 4) != 16) return LCO_ERR_FORMAT;
  const uint64_t payload_bits = get_le(s + 40, 8);
  const uint64_t total_bytes = get_le(s + 48, 8);
  if (get_le(s + 56, 8) != L.payload_off) return LCO_ERR_FORMAT;
  if (total_bytes > bytes || total_bytes < L.payload_off) return LCO_ERR_FORMAT;

  Parsed p;
  p.n = n;
  p.layout = L;
  p.payload_bits = payload_bits;
  p.total_bytes = total_bytes;
  p.table.nbits = nbits;
  p.table.nsym = static_cast<int>(nsym);
  uint64_t count_sum = 0, bit_sum = 0;
  int seen_max = 0, used = 0;
  for (uint64_t j = 0; j < nsym; ++j) {
    const uint8_t* e = s + L.table_off + 16 * j;
    p.table.key[j] = static_cast<int>(get_le(e, 2));
    p.table.len[j] = static_cast<int>(e[2]);
    p.table.rep[j] = bits_float(static_cast<uint32_t>(get_le(e + 4, 4)));
    p.table.count[j] = get_le(e + 8, 8);
    if (e[3] != 0 || p.table.len[j] > 63) return LCO_ERR_FORMAT;
    if (!fixed && !shared && p.table.count[j] == 0 && p.table.len[j] != 0) return LCO_ERR_FORMAT;
    if (p.table.count[j] > 0) used += 1;
    count_sum += p.table.count[j];
    bit_sum += p.table.count[j] * static_cast<uint64_t>(p.table.len[j]);
    seen_max = std::max(seen_max, p.table.len[j]);
  }
  if (count_sum != n || bit_sum != payload_bits || static_cast<uint64_t>(seen_max) != max_len)
    return LCO_ERR_FORMAT;
  p.table.max_len = seen_max;
  p.table.fixed = fixed;
  p.table.shared = shared;
  p.table.cached = cached;
  p.table.mean = mean;
  if (fixed) {
    int width = 0;
    while ((1ull << width) < nsym) width += 1;
    for (uint64_t j = 0; j < nsym; ++j) {
      if (p.table.len[j] != width) return LCO_ERR_FORMAT;
      p.table.code[j] = j;
    }
  } else if (shared ? seen_max != 0 : used >= 2) {
    // Kraft equality, as an exact integer sum of 2^(63-len), over the symbols that have a code: the used ones,
    // and with a shared table also those that only other parts of the larger vector use.
    unsigned __int128 kraft = 0;
    for (uint64_t j = 0; j < nsym; ++j) {
      if (shared ? p.table.len[j] == 0 : p.table.count[j] == 0) {
        if (p.table.count[j] != 0) return LCO_ERR_FORMAT;
        continue;
      }
      if (p.table.len[j] == 0) return LCO_ERR_FORMAT;
      kraft += static_cast<unsigned __int128>(1) << (63 - p.table.len[j]);
    }
    if (kraft != (static_cast<unsigned __int128>(1) << 63)) return LCO_ERR_FORMAT;
  } else if (seen_max != 0) {
    return LCO_ERR_FORMAT;
  }
  if (!fixed) canonical_codes(p.table.len, p.table.nsym, p.table.code);

  // chunk index must start at 0, be non-decreasing, 16-aligned and end at the payload size.
  const uint8_t* ci = s + L.chunk_index_off;
  uint64_t prev = 0;
  if (get_le(ci, 8) != 0) return LCO_ERR_FORMAT;
  for (uint64_t c = 1; c <= L.nchunks; ++c) {
    const uint64_t off = get_le(ci + 8 * c, 8);
    if (off < prev || off % 16 != 0) return LCO_ERR_FORMAT;
    prev = off;
  }
  if (L.payload_off + prev != total_bytes) return LCO_ERR_FORMAT;
  *out = p;
  return LCO_OK;
}

// Explicit binary code tree. child[bit][node] is 0 when absent, a node index when positive and
// -(symbol+1) at a leaf; node 0 is the root.
struct CodeTree {
  std::vector<int> child[2] = {std::vector<int>(1, 0), std::vector<int>(1, 0)};
  int only = 0;  // the symbol every element has when no code has a length (fewer than two used symbols)
};

int build_tree(const Table& t, CodeTree* tree) {
  for (int j = 0; j < t.nsym; ++j)
    if (t.count[j] > 0) tree->only = j;
  for (int j = 0; j < t.nsym; ++j) {
    if (t.len[j] == 0) continue;
    int node = 0;
    for (int b = t.len[j] - 1; b >= 0; --b) {
      const int bit = static_cast<int>((t.code[j] >> b) & 1);
      if (b == 0) {
        tree->child[bit][node] = -(j + 1);
        break;
      }
      if (tree->child[bit][node] == 0) {
        tree->child[0].push_back(0);
        tree->child[1].push_back(0);
        tree->child[bit][node] = static_cast<int>(tree->child[0].size()) - 1;
      }
      node = tree->child[bit][node];
      if (node < 0) return LCO_ERR_FORMAT;
    }
  }
  return LCO_OK;
}

// Decodes the symbols of chunk c by walking the code tree one bit at a time.
int decode_chunk(const uint8_t* s, const Parsed& p, const CodeTree& tree, uint64_t c, sym_t* sym /*[n]*/) {
  const Layout& L = p.layout;
  const uint8_t* chunk_index = s + L.chunk_index_off;
  const uint8_t* lane_index = s + L.lane_index_off;
  const uint64_t off = get_le(chunk_index + 8 * c, 8);
  const uint64_t size = get_le(chunk_index + 8 * (c + 1), 8) - off;
  const uint8_t* chunk = s + L.payload_off + off;
  uint64_t bit = 0;
  for (uint64_t lane = 0; lane < kLanes; ++lane) {
    const uint64_t lane_bits = get_le(lane_index + 2 * (kLanes * c + lane), 2);
    const uint64_t lane_end = bit + lane_bits;
    if (lane_end > 8 * size) return LCO_ERR_FORMAT;
    for (uint64_t j = 0; j < kSteps; ++j) {
      for (uint64_t e = 0; e < kGroup; ++e) {
        const uint64_t i = element_index(c, lane, j, e);
        if (i >= p.n) continue;
        int node = 0;
        while (true) {
          if (bit >= lane_end) return LCO_ERR_FORMAT;
          const int b = get_chunk_bit(chunk, bit);
          bit += 1;
          node = tree.child[b][node];
          if (node < 0) break;
          if (node == 0) return LCO_ERR_FORMAT;
        }
        sym[i] = static_cast<sym_t>(-node - 1);
      }
    }
    if (bit != lane_end) return LCO_ERR_FORMAT;
  }
  return LCO_OK;
}

// Decodes every symbol of a stream, chunk after chunk.
int decode_symbols(const uint8_t* s, uint64_t bytes, const Parsed& p, sym_t* sym /*[n]*/) {
  (void)bytes;
  CodeTree tree;
  const int rc = build_tree(p.table, &tree);
  if (rc != LCO_OK) return rc;
  if (p.table.max_len == 0) {
    for (uint64_t i = 0; i < p.n; ++i) sym[i] = static_cast<sym_t>(tree.only);
    return LCO_OK;
  }
  for (uint64_t c = 0; c < p.layout.nchunks; ++c) {
    const int rc2 = decode_chunk(s, p, tree, c, sym);
    if (rc2 != LCO_OK) return rc2;
  }
  return LCO_OK;
}

// Writes header and symbol table of a stream (format sections 3.1 and 3.2).
void write_header_and_table(uint8_t* stream, const Table& t, uint64_t n, int nbits, const Layout& L,
                            uint64_t payload_bits, uint64_t payload_bytes) {
  for (int j = 0; j < t.nsym; ++j) {
    uint8_t* e = stream + L.table_off + 16 * j;
    put_le(e, static_cast<uint64_t>(t.key[j]), 2);
    e[2] = static_cast<uint8_t>(t.len[j]);
    e[3] = 0;
    put_le(e + 4, float_bits(t.rep[j]), 4);
    put_le(e + 8, t.count[j], 8);
  }
  uint8_t* h = stream;
  h[0] = 'L'; h[1] = 'C'; h[2] = 'C'; h[3] = '1';
  put_le(h + 4, 1, 2);
  h[6] = static_cast<uint8_t>(nbits);
  h[7] = static_cast<uint8_t>(t.fixed | (t.shared << 1) | (t.cached << 2) | (t.mean << 3));
  put_le(h + 8, n, 8);
  put_le(h + 16, static_cast<uint64_t>(t.nsym), 4);
  put_le(h + 20, static_cast<uint64_t>(t.max_len), 4);
  put_le(h + 24, kChunkElems, 4);
  put_le(h + 28, kLanes, 2);
  put_le(h + 30, kGroup, 2);
  put_le(h + 32, L.nchunks, 4);
  put_le(h + 36, 16, 4);
  put_le(h + 40, payload_bits, 8);
  put_le(h + 48, L.payload_off + payload_bytes, 8);
  put_le(h + 56, L.payload_off, 8);
}

// Runs fn(t) for t in [0, nthreads) on that many threads (the timing mode that uses all host cores).
template <class F>
void run_threads(int nthreads, F fn) {
  std::vector<std::thread> pool;
  for (int t = 1; t < nthreads; ++t) pool.emplace_back(fn, t);
  fn(0);
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// Bucket statistics of the delta (Algorithm 1 step 4; Section 3.1.1). mmin/mmax are the smallest and
// largest mantissa fields in each bucket; for an empty bucket they are 0x7FFFFF and 0.
int lco_bins(const float* base, const float* cur, uint64_t n, uint64_t* count, uint32_t* mmin,
             uint32_t* mmax) {
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n, buckets.data());
  for (int k = 0; k < 512; ++k) {
    count[k] = buckets[k].count;
    if (buckets[k].count == 0) {
      mmin[k] = 0x7FFFFF;
      mmax[k] = 0;
    } else {
      const uint32_t a = float_bits(buckets[k].vmin) & 0x7FFFFF;
      const uint32_t b = float_bits(buckets[k].vmax) & 0x7FFFFF;
      mmin[k] = std::min(a, b);
      mmax[k] = std::max(a, b);
    }
  }
  return LCO_OK;
}

// Symbol table (selection, representatives, counts, code lengths, codes) for a delta vector.
// Arrays have 256 entries; returns nsym (>= 1) or a negative status.
// `fixed`: 0 for the Huffman code, 1 for fixed-width codes (format section 1.5).
int lco_table_mode(const float* base, const float* cur, uint64_t n, int nbits, int fixed, int* key, float* rep,
                   uint64_t* count, int* len, uint64_t* code) {
  if (nbits < 1 || nbits > 9 || fixed < 0 || fixed > 1) return LCO_ERR_ARG;
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n, buckets.data());
  Table t;
  const int rc = build_table(buckets.data(), n, nbits, &t, nullptr, fixed);
  if (rc != LCO_OK) return rc;
  for (int j = 0; j < t.nsym; ++j) {
    key[j] = t.key[j];
    rep[j] = t.rep[j];
    count[j] = t.count[j];
    len[j] = t.len[j];
    code[j] = t.code[j];
  }
  return t.nsym;
}

int lco_table(const float* base, const float* cur, uint64_t n, int nbits, int* key, float* rep,
              uint64_t* count, int* len, uint64_t* code) {
  return lco_table_mode(base, cur, n, nbits, 0, key, rep, count, len, code);
}

// Per-element symbol ids of the quantized delta (what the payload encodes), in element order.
int lco_symbols(const float* base, const float* cur, uint64_t n, int nbits, uint16_t* sym) {
  if (nbits < 1 || nbits > 9) return LCO_ERR_ARG;
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n, buckets.data());
  Table t;
  Selection sel;
  const int rc = build_table(buckets.data(), n, nbits, &t, &sel);
  if (rc != LCO_OK) return rc;
  for (uint64_t i = 0; i < n; ++i) sym[i] = static_cast<sym_t>(sel.symbol_of_key[bucket_key(cur[i] - base[i])]);
  return LCO_OK;
}

// Huffman lengths and canonical codes for an arbitrary count vector (exposed so the construction can
// be tested on its own against brute force).
int lco_huffman(const uint64_t* count, int nsym, int* len, uint64_t* code) {
  if (nsym < 1 || nsym > 256) return LCO_ERR_ARG;
  huffman_lengths(count, nsym, len);
  canonical_codes(len, nsym, code);
  return LCO_OK;
}

// Midrange representative of two values of one bucket.
float lco_midrange(float vmin, float vmax) { return midrange(vmin, vmax); }

// The paper's size model for fixed-width bucket indices (Section 3.1.1): n*ceil(log2 k) + k*b bits.
uint64_t lco_model_bits(uint64_t n, uint64_t k, uint64_t b) {
  uint64_t width = 0;
  while ((1ull << width) < k) width += 1;
  return n * width + k * b;
}

uint64_t lco_stream_bound(uint64_t n, int nbits) { return stream_bound(n, nbits); }

// Full compress pass: Algorithm 1 steps 4-6. Writes the stream, returns its size through *out_bytes.
// `fixed`: 0 for the Huffman code (Section 3.1.2), 1 for fixed-width bucket indices (the size model of
// Section 3.1.1 and the "E" / "E+P" stages of Section 4.3's size breakdown).
// `cache`: null, or the length cache of Section 3.2's "Huffman Code Table Caching" (read and updated).
static int compress_body(const float* base, const float* cur, uint64_t n, int nbits, int fixed, uint8_t* cache,
                         uint8_t* stream, uint64_t capacity, uint64_t* out_bytes, int mean = 0) {
  if (nbits < 1 || nbits > 9 || fixed < 0 || fixed > 1 || n >= (1ull << 32) || (cache && fixed)) return LCO_ERR_ARG;
  if (mean && (fixed || cache)) return LCO_ERR_ARG;
  if (capacity < stream_bound(n, nbits)) return LCO_ERR_CAPACITY;
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n, buckets.data());
  Table t;
  Selection sel;
  const int rc = build_table(buckets.data(), n, nbits, &t, &sel, fixed, cache, mean);
  if (rc != LCO_OK) return rc;

  const Layout L = layout_for(n, t.nsym);
  std::memset(stream, 0, L.payload_off);

  uint8_t* chunk_index = stream + L.chunk_index_off;
  uint8_t* lane_index = stream + L.lane_index_off;
  uint64_t payload_bytes = 0;
  uint64_t payload_bits = 0;
  for (uint64_t c = 0; c < L.nchunks; ++c) {
    put_le(chunk_index + 8 * c, payload_bytes, 8);
    uint64_t chunk_bits = 0;
    const uint64_t chunk_bytes = encode_chunk(base, cur, n, t, sel, c, lane_index + 2 * kLanes * c,
                                              stream + L.payload_off + payload_bytes, &chunk_bits);
    payload_bytes += chunk_bytes;
    payload_bits += chunk_bits;
  }
  put_le(chunk_index + 8 * L.nchunks, payload_bytes, 8);

  write_header_and_table(stream, t, n, nbits, L, payload_bits, payload_bytes);
  *out_bytes = L.payload_off + payload_bytes;
  return LCO_OK;
}

int lco_compress_mode(const float* base, const float* cur, uint64_t n, int nbits, int fixed, uint8_t* stream,
                      uint64_t capacity, uint64_t* out_bytes) {
  return compress_body(base, cur, n, nbits, fixed, nullptr, stream, capacity, out_bytes);
}

// Compress pass with the length cache of Section 3.2 ("Huffman Code Table Caching"); cache: 512 rows of 512 bytes.
int lco_compress_cached(const float* base, const float* cur, uint64_t n, int nbits, uint8_t* cache, uint8_t* stream,
                        uint64_t capacity, uint64_t* out_bytes) {
  if (!cache) return LCO_ERR_ARG;
  return compress_body(base, cur, n, nbits, 0, cache, stream, capacity, out_bytes);
}

// Compress pass with bucket means as representatives (format section 1.8) instead of Section 3.1.1's midrange.
int lco_compress_mean(const float* base, const float* cur, uint64_t n, int nbits, uint8_t* stream, uint64_t capacity,
                      uint64_t* out_bytes) {
  return compress_body(base, cur, n, nbits, 0, nullptr, stream, capacity, out_bytes, 1);
}

// The mean of `count` values that share sign and exponent (one bucket), as the mean variant represents them.
// Returns NaN if they do not form one bucket of normal numbers.
float lco_bucket_mean(const float* values, uint64_t count) {
  if (count == 0) return NAN;
  std::vector<float> zero(count, 0.0f);
  std::vector<Bucket> buckets(512);
  delta_buckets(zero.data(), values, count, buckets.data());
  const int key = bucket_key(values[0] - 0.0f);
  if (buckets[key].count != count || (key & 255) == 0 || (key & 255) == 255) return NAN;
  return bucket_mean(key, buckets[key].sig_sum, count);
}

// The caching step alone: code lengths of `nsym` symbols with the given counts (n = their sum). Returns 1 on a hit.
int lco_cached_lengths(const uint64_t* count, int nsym, int nbits, uint64_t n, uint8_t* cache, int* len) {
  return cached_lengths(count, nsym, nbits, n, cache, len);
}

int lco_compress(const float* base, const float* cur, uint64_t n, int nbits, uint8_t* stream,
                 uint64_t capacity, uint64_t* out_bytes) {
  return lco_compress_mode(base, cur, n, nbits, 0, stream, capacity, out_bytes);
}

// Symbol ids stored in a stream, in element order (decode only, no arithmetic).
int lco_decode_symbols(const uint8_t* stream, uint64_t bytes, uint64_t n, uint16_t* sym) {
  Parsed p;
  const int rc = parse_stream(stream, bytes, &p);
  if (rc != LCO_OK) return rc;
  if (p.n != n) return LCO_ERR_MISMATCH;
  return decode_symbols(stream, bytes, p, sym);
}

// Recovery: out = ((base + d_1) + d_2) + ... + d_k in fp32, stream order (Algorithm 1 step 7 applied
// k times; the reconstruction identity u_t = u_0 + sum of the quantized deltas).
int lco_recover(const float* base, const uint8_t* const* streams, const uint64_t* stream_bytes, int k,
                uint64_t n, float* out) {
  if (k < 1) return LCO_ERR_ARG;
  std::vector<Parsed> parsed(static_cast<size_t>(k));
  for (int j = 0; j < k; ++j) {
    const int rc = parse_stream(streams[j], stream_bytes[j], &parsed[j]);
    if (rc != LCO_OK) return rc;
    if (parsed[j].n != n) return LCO_ERR_MISMATCH;
  }
  std::vector<float> x(base, base + n);
  std::vector<sym_t> sym(n);
  for (int j = 0; j < k; ++j) {
    const int rc = decode_symbols(streams[j], stream_bytes[j], parsed[j], sym.data());
    if (rc != LCO_OK) return rc;
    for (uint64_t i = 0; i < n; ++i) x[i] = x[i] + parsed[j].table.rep[sym[i]];
  }
  for (uint64_t i = 0; i < n; ++i) out[i] = x[i];
  return LCO_OK;
}

// Algorithm 1 step 7 computed directly, without a bitstream: out = base + quantized(cur - base).
int lco_apply_quantized(const float* base, const float* cur, uint64_t n, int nbits, float* out) {
  if (nbits < 1 || nbits > 9) return LCO_ERR_ARG;
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n, buckets.data());
  Table t;
  Selection sel;
  const int rc = build_table(buckets.data(), n, nbits, &t, &sel);
  if (rc != LCO_OK) return rc;
  for (uint64_t i = 0; i < n; ++i) out[i] = base[i] + t.rep[sel.symbol_of_key[bucket_key(cur[i] - base[i])]];
  return LCO_OK;
}

// Codes only the listed chunks of the stream that lco_compress would write for the whole vector (the
// table comes from the whole vector). For chunk m: lane_bits[32*m ..] and bytes[m] payload bytes at
// payload + m*stride. Lets a test check chunks of a vector too large to code in full.
int lco_compress_chunks(const float* base, const float* cur, uint64_t n, int nbits, const uint64_t* chunk_ids,
                        uint64_t m, uint16_t* lane_bits, uint8_t* payload, uint64_t stride, uint64_t* bytes) {
  if (nbits < 1 || nbits > 9) return LCO_ERR_ARG;
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n, buckets.data());
  Table t;
  Selection sel;
  const int rc = build_table(buckets.data(), n, nbits, &t, &sel);
  if (rc != LCO_OK) return rc;
  std::vector<uint8_t> chunk(kChunkElems * 8 + 16);
  for (uint64_t k = 0; k < m; ++k) {
    uint8_t li[64];
    uint64_t bits = 0;
    const uint64_t sz = encode_chunk(base, cur, n, t, sel, chunk_ids[k], li, chunk.data(), &bits);
    if (sz > stride) return LCO_ERR_CAPACITY;
    for (int lane = 0; lane < 32; ++lane) lane_bits[32 * k + lane] = static_cast<uint16_t>(get_le(li + 2 * lane, 2));
    std::memcpy(payload + k * stride, chunk.data(), sz);
    bytes[k] = sz;
  }
  return LCO_OK;
}


// Checkpoint merging (Section 3.2, "Checkpoint Merging"): k consecutive checkpoints become one
// super-step checkpoint. The paper does not say how the merged checkpoint is coded; the reading taken
// here is the scheme applied once more to the summed change: the state the k streams recover is
// compressed against the same base,
//   merged = compress(base, recover(base, streams)).
// The merged stream therefore quantizes a second time: recovering it gives a state within the
// quantization error of, not bit-identical to, what the k streams recover.
int lco_merge(const float* base, const uint8_t* const* streams, const uint64_t* stream_bytes, int k, uint64_t n,
              int nbits, uint8_t* stream, uint64_t capacity, uint64_t* out_bytes) {
  std::vector<float> recovered(n);
  const int rc = lco_recover(base, streams, stream_bytes, k, n, recovered.data());
  if (rc != LCO_OK) return rc;
  return lco_compress(base, recovered.data(), n, nbits, stream, capacity, out_bytes);
}

// ---- the same two passes on several host threads (timing mode: "all host cores") -----------------
// The steps are those of lco_compress / lco_recover; only the loops over elements and chunks are split
// into contiguous ranges, one per thread. Bucket statistics merge by sum / min / max; chunks are coded
// and decoded independently once the table is known. The results are byte-identical to the
// single-threaded functions (a test checks that).

int lco_compress_mode_mt(const float* base, const float* cur, uint64_t n, int nbits, int fixed, uint8_t* stream,
                         uint64_t capacity, uint64_t* out_bytes, int nthreads) {
  if (nbits < 1 || nbits > 9 || fixed < 0 || fixed > 1 || n >= (1ull << 32) || nthreads < 1) return LCO_ERR_ARG;
  if (capacity < stream_bound(n, nbits)) return LCO_ERR_CAPACITY;
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  auto range = [&](int t, uint64_t total) {
    return std::pair<uint64_t, uint64_t>(total * t / nthreads, total * (t + 1) / nthreads);
  };
  // statistics: one set of buckets per thread over a range of whole chunks, then merged
  std::vector<std::vector<Bucket>> part(nthreads, std::vector<Bucket>(512));
  run_threads(nthreads, [&](int t) {
    const auto r = range(t, nchunks);
    const uint64_t lo = std::min(n, r.first * kChunkElems), hi = std::min(n, r.second * kChunkElems);
    delta_buckets(base + lo, cur + lo, hi - lo, part[t].data());
  });
  std::vector<Bucket> buckets(512);
  for (int t = 0; t < nthreads; ++t)
    for (int key = 0; key < 512; ++key) {
      const Bucket& b = part[t][key];
      Bucket& m = buckets[key];
      if (b.count == 0) continue;
      if (m.count == 0) {
        m = b;
      } else {
        m.count += b.count;
        m.sig_sum += b.sig_sum;
        if (b.vmin < m.vmin) m.vmin = b.vmin;
        if (b.vmax > m.vmax) m.vmax = b.vmax;
      }
    }
  Table t;
  Selection sel;
  const int rc = build_table(buckets.data(), n, nbits, &t, &sel, fixed);
  if (rc != LCO_OK) return rc;
  const Layout L = layout_for(n, t.nsym);
  std::memset(stream, 0, L.payload_off);
  // every chunk coded into a buffer of its own, then laid out in order
  std::vector<std::vector<uint8_t>> coded(nchunks);
  std::vector<uint64_t> bits(nchunks, 0);
  uint8_t* lane_index = stream + L.lane_index_off;
  run_threads(nthreads, [&](int th) {
    const auto r = range(th, nchunks);
    std::vector<uint8_t> chunk(kChunkElems * 8 + 16);
    for (uint64_t c = r.first; c < r.second; ++c) {
      const uint64_t sz = encode_chunk(base, cur, n, t, sel, c, lane_index + 2 * kLanes * c, chunk.data(), &bits[c]);
      coded[c].assign(chunk.begin(), chunk.begin() + sz);
    }
  });
  uint8_t* chunk_index = stream + L.chunk_index_off;
  uint64_t payload_bytes = 0, payload_bits = 0;
  for (uint64_t c = 0; c < nchunks; ++c) {
    put_le(chunk_index + 8 * c, payload_bytes, 8);
    std::memcpy(stream + L.payload_off + payload_bytes, coded[c].data(), coded[c].size());
    payload_bytes += coded[c].size();
    payload_bits += bits[c];
  }
  put_le(chunk_index + 8 * nchunks, payload_bytes, 8);
  write_header_and_table(stream, t, n, nbits, L, payload_bits, payload_bytes);
  *out_bytes = L.payload_off + payload_bytes;
  return LCO_OK;
}

int lco_compress_mt(const float* base, const float* cur, uint64_t n, int nbits, uint8_t* stream,
                    uint64_t capacity, uint64_t* out_bytes, int nthreads) {
  return lco_compress_mode_mt(base, cur, n, nbits, 0, stream, capacity, out_bytes, nthreads);
}

int lco_recover_mt(const float* base, const uint8_t* const* streams, const uint64_t* stream_bytes, int k,
                   uint64_t n, float* out, int nthreads) {
  if (k < 1 || nthreads < 1) return LCO_ERR_ARG;
  std::vector<Parsed> parsed(static_cast<size_t>(k));
  std::vector<CodeTree> trees(static_cast<size_t>(k));
  for (int j = 0; j < k; ++j) {
    int rc = parse_stream(streams[j], stream_bytes[j], &parsed[j]);
    if (rc != LCO_OK) return rc;
    if (parsed[j].n != n) return LCO_ERR_MISMATCH;
    if ((rc = build_tree(parsed[j].table, &trees[j])) != LCO_OK) return rc;
  }
  const uint64_t nchunks = (n + kChunkElems - 1) / kChunkElems;
  std::vector<sym_t> sym(n);
  std::vector<int> status(nthreads, LCO_OK);
  for (uint64_t i = 0; i < n; ++i) out[i] = base[i];
  for (int j = 0; j < k; ++j) {
    run_threads(nthreads, [&](int th) {
      const uint64_t c0 = nchunks * th / nthreads, c1 = nchunks * (th + 1) / nthreads;
      for (uint64_t c = c0; c < c1; ++c) {
        const uint64_t lo = c * kChunkElems, hi = std::min(n, lo + kChunkElems);
        if (parsed[j].table.max_len == 0) {
          for (uint64_t i = lo; i < hi; ++i) sym[i] = static_cast<sym_t>(trees[j].only);
        } else {
          const int rc = decode_chunk(streams[j], parsed[j], trees[j], c, sym.data());
          if (rc != LCO_OK) status[th] = rc;
        }
        for (uint64_t i = lo; i < hi; ++i) out[i] = out[i] + parsed[j].table.rep[sym[i]];
      }
    });
    for (int th = 0; th < nthreads; ++th)
      if (status[th] != LCO_OK) return status[th];
  }
  return LCO_OK;
}


// One shard of a vector that is split over several devices (format section 1.6): the table (kept buckets,
// representatives, code) comes from the statistics of the WHOLE vector [0, n_total), which every shard obtains by
// exchanging its 512 bucket statistics (counts add, minima and maxima combine), so all shards code with the same
// table; the stream codes the elements [lo, hi) only, as a vector of hi - lo elements, and its table lists the
// shard's own counts. Recovering every shard's stream over its part of the base gives, part by part, what the
// stream of the whole vector recovers.
int lco_compress_shard(const float* base, const float* cur, uint64_t n_total, uint64_t lo, uint64_t hi, int nbits,
                       uint8_t* stream, uint64_t capacity, uint64_t* out_bytes) {
  if (nbits < 1 || nbits > 9 || n_total >= (1ull << 32) || lo > hi || hi > n_total) return LCO_ERR_ARG;
  const uint64_t n = hi - lo;
  if (capacity < stream_bound(n, nbits)) return LCO_ERR_CAPACITY;
  std::vector<Bucket> buckets(512);
  delta_buckets(base, cur, n_total, buckets.data());
  Table t;
  Selection sel;
  const int rc = build_table(buckets.data(), n_total, nbits, &t, &sel);
  if (rc != LCO_OK) return rc;
  t.shared = 1;
  for (int j = 0; j < t.nsym; ++j) t.count[j] = 0;
  for (uint64_t i = lo; i < hi; ++i) t.count[sel.symbol_of_key[bucket_key(cur[i] - base[i])]] += 1;

  const Layout L = layout_for(n, t.nsym);
  std::memset(stream, 0, L.payload_off);
  uint8_t* chunk_index = stream + L.chunk_index_off;
  uint8_t* lane_index = stream + L.lane_index_off;
  uint64_t payload_bytes = 0, payload_bits = 0;
  for (uint64_t c = 0; c < L.nchunks; ++c) {
    put_le(chunk_index + 8 * c, payload_bytes, 8);
    uint64_t chunk_bits = 0;
    payload_bytes += encode_chunk(base + lo, cur + lo, n, t, sel, c, lane_index + 2 * kLanes * c,
                                  stream + L.payload_off + payload_bytes, &chunk_bits);
    payload_bits += chunk_bits;
  }
  put_le(chunk_index + 8 * L.nchunks, payload_bytes, 8);
  write_header_and_table(stream, t, n, nbits, L, payload_bits, payload_bytes);
  *out_bytes = L.payload_off + payload_bytes;
  return LCO_OK;
}

}  // extern "C"
