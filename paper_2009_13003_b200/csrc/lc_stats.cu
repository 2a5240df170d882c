// Statistics pass: fused delta, (sign, exponent) key extraction, 512-bin histogram with per-bin
// minimum / maximum, and the 1-byte-per-element key plane for the encode pass.
//
// Paper: Algorithm 1 step 4 (delta against the tracked state) and Section 3.1.1, exponent-based
// quantization (bucket = identical sign and exponent; representative from the bucket's min and max).
//
// Bound: HBM. 8 bytes per element must be read; 1 byte per element is written.
//
// Two settings decide whether the pass reaches that bound. (1) The L1 cache: a kernel with this much dynamic
// shared memory gets the largest shared-memory carve-out by default, and the small L1 that is left cannot keep
// enough loads in flight (the pass then runs 15 % slower). The launcher asks for just the carve-out its
// resident CTAs need. (2) Plain cached loads (ld.global.nc): with the L1 available they are faster than loads
// that bypass it. Two CTAs of 12 warps per SM share 2 x 68 KB of tables; three CTAs of 8 warps would need a
// carve-out that leaves no L1.
//
// Design for a skewed histogram (a handful of exponents hold almost all elements):
//  * counts live in shared memory as cnt[slot][lane] (slot = the key with the sign moved to bit 0):
//    every lane of a warp owns its own column, so the
//    32 atomics of one warp instruction always hit 32 different banks and never the same address,
//    whatever the keys are;
//  * min / max are kept per key as a pair of running maxima (of ~bits and of bits: inside one key the
//    order of the bit patterns is the order of the mantissas). A lane first reads the pair with a
//    plain load and only issues an atomic when its value would improve it, which after the first few
//    elements almost never happens;
//  * counts are integers and min / max are order-free, so the result is deterministic.
#include "lc_common.cuh"

namespace lc {
namespace {

constexpr int kStatsThreads = 384;
constexpr int kRows = 8;  // steps per unit
constexpr uint32_t kCntWords = kKeys * 32;
constexpr uint32_t kStatsSmem = (kCntWords + 2 * kKeys) * 4;  // 64 KB + 4 KB
// Mean-representative variant (format section 1.8): two more tables of the same shape hold, per key and lane, the
// sums of the low 12 and of the high 11 bits of the mantissa fields. A column receives at most 32 elements per warp
// and unit, so 32-bit sums hold for kMeanMaxUnitsPerWarp units per warp: 12 warps * 32 * 4095 * 2731 < 2^32.
constexpr uint32_t kStatsSmemMean = (3 * kCntWords + 2 * kKeys) * 4;  // 192 KB + 4 KB: one CTA per SM
constexpr uint64_t kMeanMaxUnitsPerWarp = 2731;

__device__ __forceinline__ float4 ld_stream(const float4* p) {
  float4 v;
  asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p));
  return v;
}

// Slot of a delta's bucket in the shared-memory tables: (exponent field << 1) | sign. The two signs of one
// exponent are neighbours and 8 consecutive exponents fill the 16 bank pairs of a 64-bit access exactly once,
// so the few hot buckets of a vector (neighbouring exponents, both signs) rarely meet in a bank. The low byte
// of the slot is the element's byte in the key plane.
__device__ __forceinline__ uint32_t slot_of(uint32_t bits) { return ((bits >> 22) & 0x1FEu) | (bits >> 31); }
__device__ __forceinline__ uint32_t key_of_slot(uint32_t slot) { return ((slot & 1u) << 8) | (slot >> 1); }

template <bool MEAN>
struct Acc {
  uint32_t* cnt_lane;  // &cnt[lane]
  uint2* mm;
  __device__ __forceinline__ void sum(uint32_t bits, uint32_t slot) {
    if (MEAN) {
      atomicAdd(cnt_lane + kCntWords + slot * 32, bits & 0xFFFu);
      atomicAdd(cnt_lane + 2 * kCntWords + slot * 32, (bits >> 12) & 0x7FFu);
    }
  }
  __device__ __forceinline__ void improve(uint32_t bits, uint32_t slot, uint2 cur) {
    if (~bits > cur.x) atomicMax(&mm[slot].x, ~bits);
    if (bits > cur.y) atomicMax(&mm[slot].y, bits);
  }
  __device__ __forceinline__ void add(uint32_t bits) {
    const uint32_t slot = slot_of(bits);
    atomicAdd(cnt_lane + slot * 32, 1u);
    sum(bits, slot);
    improve(bits, slot, mm[slot]);
  }
  // Four elements at once: the four reads of the running min / max pairs go out together, and one test
  // covers all eight comparisons, because after the first few elements none of them ever holds.
  __device__ __forceinline__ void add4(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t d3, uint32_t k0, uint32_t k1,
                                       uint32_t k2, uint32_t k3) {
    const uint2 c0 = mm[k0], c1 = mm[k1], c2 = mm[k2], c3 = mm[k3];
    atomicAdd(cnt_lane + k0 * 32, 1u);
    atomicAdd(cnt_lane + k1 * 32, 1u);
    atomicAdd(cnt_lane + k2 * 32, 1u);
    atomicAdd(cnt_lane + k3 * 32, 1u);
    sum(d0, k0);
    sum(d1, k1);
    sum(d2, k2);
    sum(d3, k3);
    const bool any = (~d0 > c0.x) | (d0 > c0.y) | (~d1 > c1.x) | (d1 > c1.y) | (~d2 > c2.x) | (d2 > c2.y) |
                     (~d3 > c3.x) | (d3 > c3.y);
    if (any) {
      improve(d0, k0, c0);
      improve(d1, k1, c1);
      improve(d2, k2, c2);
      improve(d3, k3, c3);
    }
  }
};

template <bool MEAN>
__global__ void __launch_bounds__(kStatsThreads, MEAN ? 1 : 2)
stats_kernel(const float* __restrict__ base, const float* __restrict__ cur, uint64_t n, uint64_t nunits,
             Control* __restrict__ ctl, uint8_t* __restrict__ plane) {
  extern __shared__ __align__(16) uint32_t smem[];
  // MEAN: cnt, then the two sum tables, then mm
  constexpr uint32_t kTables = MEAN ? 3 : 1;
  uint32_t* cnt = smem;
  uint2* mm = reinterpret_cast<uint2*>(smem + kTables * kCntWords);
  for (uint32_t i = threadIdx.x; i < kTables * kCntWords + 2 * kKeys; i += kStatsThreads) smem[i] = 0;
  __syncthreads();

  const uint32_t lane = threadIdx.x & 31;
  const uint64_t warp = (uint64_t)blockIdx.x * (kStatsThreads / 32) + (threadIdx.x >> 5);
  const uint64_t nwarps = (uint64_t)gridDim.x * (kStatsThreads / 32);
  Acc<MEAN> acc{cnt + lane, mm};

  for (uint64_t u = warp; u < nunits; u += nwarps) {
    const uint64_t i0 = u * kUnitElems;
    uint32_t ew[kRows];
    if (i0 + kUnitElems <= n) {
      const float4* b4 = reinterpret_cast<const float4*>(base + i0) + lane;
      const float4* c4 = reinterpret_cast<const float4*>(cur + i0) + lane;
      float4 b[kRows], c[kRows];
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        b[r] = ld_stream(b4 + 32 * r);
        c[r] = ld_stream(c4 + 32 * r);
      }
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const uint32_t d0 = __float_as_uint(__fsub_rn(c[r].x, b[r].x));
        const uint32_t d1 = __float_as_uint(__fsub_rn(c[r].y, b[r].y));
        const uint32_t d2 = __float_as_uint(__fsub_rn(c[r].z, b[r].z));
        const uint32_t d3 = __float_as_uint(__fsub_rn(c[r].w, b[r].w));
        const uint32_t k0 = slot_of(d0), k1 = slot_of(d1), k2 = slot_of(d2), k3 = slot_of(d3);
        acc.add4(d0, d1, d2, d3, k0, k1, k2, k3);
        // plane byte = low byte of the slot; gather the four into one word, element e in byte e.
        const uint32_t lo = __byte_perm(k0, k1, 0x0040);
        const uint32_t hi = __byte_perm(k2, k3, 0x0040);
        ew[r] = __byte_perm(lo, hi, 0x5410);
      }
    } else {
      // ragged tail: the last units of the vector, element by element.
#pragma unroll 1
      for (int r = 0; r < kRows; ++r) {
        uint32_t word = 0;
        for (int e = 0; e < 4; ++e) {
          const uint64_t i = i0 + 128 * r + 4 * lane + e;
          uint32_t d = 0;
          if (i < n) {
            d = __float_as_uint(__fsub_rn(cur[i], base[i]));
            acc.add(d);
          }
          word |= (slot_of(d) & 255u) << (8 * e);
        }
        ew[r] = word;
      }
    }
    uint4* ep = reinterpret_cast<uint4*>(plane + i0) + lane;
    ep[0] = make_uint4(ew[0], ew[1], ew[2], ew[3]);
    ep[32] = make_uint4(ew[4], ew[5], ew[6], ew[7]);
  }
  __syncthreads();

  // fold the 32 lane columns of each key and merge into the global bins.
  for (uint32_t slot = threadIdx.x; slot < kKeys; slot += kStatsThreads) {
    uint32_t total = 0;
#pragma unroll 8
    for (uint32_t l = 0; l < 32; ++l) total += cnt[slot * 32 + ((l + threadIdx.x) & 31)];
    if (total != 0) {
      const uint32_t key = key_of_slot(slot);
      atomicAdd(&ctl->count[key], (unsigned long long)total);
      atomicMax(&ctl->inv_min[key], mm[slot].x);
      atomicMax(&ctl->max_bits[key], mm[slot].y);
      if (MEAN) {
        unsigned long long lo = 0, hi = 0;
        for (uint32_t l = 0; l < 32; ++l) {
          lo += cnt[kCntWords + slot * 32 + ((l + threadIdx.x) & 31)];
          hi += cnt[2 * kCntWords + slot * 32 + ((l + threadIdx.x) & 31)];
        }
        atomicAdd(&ctl->mant_sum[key], lo + (hi << 12));
      }
    }
  }
}

}  // namespace

cudaError_t launch_stats(const float* base, const float* cur, uint64_t n, Control* ctl, uint8_t* plane,
                         cudaStream_t cs, bool mean) {
  const WorkspaceLayout W = workspace_layout(n);
  if (W.nunits == 0) return cudaSuccess;
  static int blocks_per_sm[kMaxDevices][2] = {}, sms[kMaxDevices] = {};  // by device ordinal and kernel variant
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  const int v = mean ? 1 : 0;
  const uint32_t smem = mean ? kStatsSmemMean : kStatsSmem;
  const void* fn = mean ? reinterpret_cast<const void*>(stats_kernel<true>) : reinterpret_cast<const void*>(stats_kernel<false>);
  if (blocks_per_sm[dev][v] == 0) {
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int nsm = 0;
    if ((e = cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    int bps = 0;
    e = mean ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, stats_kernel<true>, kStatsThreads, smem)
             : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, stats_kernel<false>, kStatsThreads, smem);
    if (e != cudaSuccess) return e;
    if (bps < 1) bps = 1;
    // carve-out in percent of the SM's 228 KB: the resident CTAs' shared memory (plus 1 KB each that the system
    // reserves), rounded up
    const int carve = (int)(((uint64_t)bps * (smem + 1024) * 100 + 228 * 1024 - 1) / (228 * 1024)) + 1;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, carve < 100 ? carve : 100);
    if (e != cudaSuccess) return e;
    sms[dev] = nsm;
    blocks_per_sm[dev][v] = bps;
  }
  const uint64_t want = (W.nunits + kStatsThreads / 32 - 1) / (kStatsThreads / 32);
  const uint64_t full = (uint64_t)sms[dev] * blocks_per_sm[dev][v];
  const unsigned grid = (unsigned)(want < full ? want : full);
  if (mean) {
    // the 32-bit column sums of the variant hold for a bounded number of units per warp (see kMeanMaxUnitsPerWarp)
    const uint64_t nwarps = (uint64_t)grid * (kStatsThreads / 32);
    if ((W.nunits + nwarps - 1) / nwarps > kMeanMaxUnitsPerWarp) return cudaErrorInvalidConfiguration;
    stats_kernel<true><<<grid, kStatsThreads, smem, cs>>>(base, cur, n, W.nunits, ctl, plane);
  } else {
    stats_kernel<false><<<grid, kStatsThreads, smem, cs>>>(base, cur, n, W.nunits, ctl, plane);
  }
  return cudaGetLastError();
}

}  // namespace lc
