// Pieces shared by the two decode kernels: shared-memory access by 32-bit address, asynchronous copies, and a
// lane's bit reader over one chunk of one stream (format section 2: a chunk is a string of bits stored in 32-bit
// words, most significant bit first; lane t's codes are a contiguous run of that string).
#pragma once

#include "lc_common.cuh"

namespace lc {
namespace dec {

constexpr uint32_t kSmemPerSm = 227 * 1024;  // usable shared memory of one CTA on sm_100
constexpr uint32_t kOverrunBytes = 512;      // padding behind the last staging area (see LaneBits::refill)

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t load_le(const uint8_t* p, int bytes) {
  uint64_t v = 0;
  for (int b = 0; b < bytes; ++b) v |= (uint64_t)p[b] << (8 * b);
  return v;
}

// ---- shared-memory access by 32-bit shared address (keeps the hot loops free of generic addressing)
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
// 16-byte load of base; volatile so that it stays where it is written (early in the loop body). A plain cached
// load (measured a few percent faster than the streaming forms with one stream, the same with four), and not
// the read-only path: `out` may be `base`, i.e. the kernel may write the memory it reads here.
__device__ __forceinline__ float4 ldg_stream_v4(const float* p) {
  float4 v;
  asm volatile("ld.global.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// Where a chunk's words are read from.
struct Source {
  const uint32_t* g;  // chunk words in global memory
  uint32_t nw;        // words in the chunk
  uint32_t sbase;     // staged: shared address of the chunk's first word
  uint32_t slim;      // staged: shared address of the last readable word (zero slack after the chunk)
};

// A lane's read state in one stream: `cnt` valid bits at the top of hi:lo (the bits below are zero).
// STAGED: the chunk's words are in the warp's staging area and `next` is the shared address of the next
// word to load. Otherwise (a chunk too large to stage) they are read from global memory and `next` is a
// word index.
template <bool STAGED>
struct LaneBits {
  uint32_t hi, lo;
  int cnt;
  uint32_t next;

  // word `idx` of the chunk, 0 beyond its end
  __device__ __forceinline__ static uint32_t word(const Source& W, uint32_t idx) {
    if (STAGED) return lds_u32(min(W.sbase + idx * 4u, W.slim));
    return idx < W.nw ? __ldg(W.g + idx) : 0u;
  }
  __device__ __forceinline__ uint32_t bitpos(const Source& W) const {
    return (STAGED ? (next - W.sbase) * 8u : next * 32u) - (uint32_t)cnt;
  }
  __device__ __forceinline__ void seek(const Source& W, uint32_t pos) {
    const uint32_t idx = pos >> 5, sh = pos & 31;
    const uint32_t w0 = word(W, idx), w1 = word(W, idx + 1);
    hi = __funnelshift_l(w1, w0, sh);
    lo = w1 << sh;
    cnt = 64 - (int)sh;
    next = STAGED ? min(W.sbase + (idx + 2) * 4u, W.slim) : idx + 2;
  }
  // Tops the buffer up with one word if 32 bits or fewer are left; afterwards cnt >= 33. All predicated.
  // STAGED: the load is not clamped: between two seeks (which do clamp) `next` moves by at most 64 words,
  // and the kernel's shared memory ends with kOverrunBytes of padding, so a damaged stream can make a lane
  // read stale shared memory but never leave the allocation.
  __device__ __forceinline__ void refill(const Source& W) {
    if (STAGED) {
      asm volatile(
          "{\n\t"
          ".reg .pred q;\n\t"
          ".reg .u32 w, t;\n\t"
          "setp.le.s32 q, %2, 32;\n\t"
          "@q ld.shared.u32 w, [%3];\n\t"
          "@q shf.r.clamp.b32 t, w, 0, %2;\n\t"   // high word of (w:0) >> cnt, i.e. w >> cnt (0 when cnt == 32)
          "@q or.b32 %0, %0, t;\n\t"
          "@q shf.r.clamp.b32 %1, 0, w, %2;\n\t"  // low word of (w:0) >> cnt; lo was 0 because cnt <= 32
          "@q add.s32 %2, %2, 32;\n\t"
          "@q add.u32 %3, %3, 4;\n\t"
          "}"
          : "+r"(hi), "+r"(lo), "+r"(cnt), "+r"(next));
    } else {
      asm volatile(
          "{\n\t"
          ".reg .pred q, r;\n\t"
          ".reg .u32 w, t;\n\t"
          ".reg .u64 a;\n\t"
          "setp.le.s32 q, %2, 32;\n\t"
          "setp.lt.and.u32 r, %3, %5, q;\n\t"     // words beyond the chunk read as 0
          "mov.u32 w, 0;\n\t"
          "mad.wide.u32 a, %3, 4, %4;\n\t"
          "@r ld.global.nc.u32 w, [a];\n\t"
          "@q shf.r.clamp.b32 t, w, 0, %2;\n\t"
          "@q or.b32 %0, %0, t;\n\t"
          "@q shf.r.clamp.b32 %1, 0, w, %2;\n\t"
          "@q add.s32 %2, %2, 32;\n\t"
          "@q add.u32 %3, %3, 1;\n\t"
          "}"
          : "+r"(hi), "+r"(lo), "+r"(cnt), "+r"(next)
          : "l"(W.g), "r"(W.nw));
    }
  }
  __device__ __forceinline__ void consume(uint32_t len) {
    hi = __funnelshift_l(lo, hi, len);
    lo <<= len;
    cnt -= (int)len;
  }
};

}  // namespace dec
}  // namespace lc
