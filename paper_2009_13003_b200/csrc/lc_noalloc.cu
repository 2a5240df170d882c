// lc_compress_noalloc: the compress pass for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc (or any allocating routine) at the point where
// they take a snapshot: a training process whose memory pool already owns the whole device, code that
// runs inside a region where allocation is forbidden or would synchronise the device, or a plug-in
// that was handed raw pointers and nothing else. lc_compress needs a scratch workspace from its
// caller; this entry point brings its own instead: a fixed array in device memory that is part of the
// library image. The price is a size limit and no concurrency (see include/lc.h).
#include "lc_common.cuh"

using namespace lc;

namespace {

// Largest vector the built-in scratch serves, and the scratch itself. The array lives in every
// device context that loads the library, from load to exit.
constexpr uint64_t kNoAllocMaxN = LC_NOALLOC_MAX_N;
constexpr uint64_t kNoAllocBytes = workspace_layout(kNoAllocMaxN).total;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// In host code the name above is only a handle; the device address has to be asked for, once per
// device, with that device current.
void* g_scratch_addr[kMaxDevices] = {};

int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LC_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return LC_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return LC_OK;
}

}  // namespace

extern "C" int lc_compress_noalloc(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                                   uint64_t stream_capacity, lc_cuda_stream_t cs) {
  if (nbits < 1 || nbits > kMaxNbits) return LC_ERR_ARG;
  if (n > kNoAllocMaxN) return LC_ERR_CAPACITY;  // beyond the built-in scratch: use lc_compress
  if (!stream || (n > 0 && (!base || !cur))) return LC_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(base) | reinterpret_cast<uintptr_t>(cur) | reinterpret_cast<uintptr_t>(stream)) & 15)
    return LC_ERR_ARG;
  if (stream_capacity < lc_stream_bound(n, nbits)) return LC_ERR_CAPACITY;
  const WorkspaceLayout W = workspace_layout(n);
  if (W.total > kNoAllocBytes) return LC_ERR_CAPACITY;

  void* scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc != LC_OK) return rc;
  uint8_t* w = static_cast<uint8_t*>(scratch);
  Control* ctl = reinterpret_cast<Control*>(w + W.control_off);
  unsigned long long* tiles = reinterpret_cast<unsigned long long*>(w + W.tiles_off);
  uint8_t* plane = w + W.plane_off;

  // the array keeps what the previous call left: counters, bins and tile descriptors must start at zero
  if (cudaMemsetAsync(w, 0, W.plane_off, cs) != cudaSuccess) return LC_ERR_CUDA;
  if (launch_stats(base, cur, n, ctl, plane, cs) != cudaSuccess) return LC_ERR_CUDA;
  if (launch_table(ctl, n, nbits, static_cast<uint8_t*>(stream), true, false, nullptr, nullptr, cs) != cudaSuccess) return LC_ERR_CUDA;
  if (launch_encode(ctl, tiles, plane, base, cur, n, static_cast<uint8_t*>(stream), nullptr, EncodeOptions(), cs) != cudaSuccess)
    return LC_ERR_CUDA;
  int32_t status = 0;
  if (cudaMemcpyAsync(&status, &ctl->status, sizeof status, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
    return LC_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return LC_ERR_CUDA;
  return status;
}
