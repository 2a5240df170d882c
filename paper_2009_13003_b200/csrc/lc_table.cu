// Table pass: one CTA turns the 512 bucket statistics into the symbol table of the stream.
//
// Paper: Section 3.1.1 (priority promotion: keep the 2^x - 1 occupied buckets with the largest
// exponent, merge the rest into one bucket of value 0; representative = average of the bucket's
// minimum and maximum) and Section 3.1.2 (Huffman code over the bucket indices). Tie-breaks and the
// canonical code assignment are those of the stream format text, sections 1.2-1.4.
//
// Latency-only: O(512) work. Writes the stream header and symbol table, and the per-key encode table
// the encode pass looks codes up in.
#include "lc_table.cuh"

namespace lc {
namespace {

__global__ void __launch_bounds__(kTableThreads)
table_kernel(Control* __restrict__ ctl, uint64_t n, int nbits, uint8_t* __restrict__ stream, int wide_ok,
             int fixed, const ShardStats* __restrict__ whole, uint8_t* __restrict__ cache, int mean) {
  table_pass(ctl, n, nbits, stream, wide_ok, fixed, whole, cache, mean);
}

}  // namespace

cudaError_t launch_table(Control* ctl, uint64_t n, int nbits, uint8_t* stream, bool wide_ok, bool fixed,
                         const ShardStats* whole, uint8_t* cache, cudaStream_t cs, bool mean) {
  table_kernel<<<1, kTableThreads, 0, cs>>>(ctl, n, nbits, stream, wide_ok ? 1 : 0, fixed ? 1 : 0, whole, cache,
                                            mean ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace lc
