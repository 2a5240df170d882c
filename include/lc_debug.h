/*
 * lc_debug.h - test and profiling aids of the LC-Checkpoint library. Not part of the product interface
 * (include/lc.h): stage dumps that the parity tests compare with the CPU oracle, per-kernel timing for
 * the benchmark, and a way to make the encode pass's bounded wait run out without hanging anything.
 * Conventions as in lc.h.
 */
#ifndef LC_DEBUG_H_
#define LC_DEBUG_H_

#include "lc.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * lc_compress (Algorithm 1 steps 4-6) with per-kernel timing: same arguments and result, but the call
 * records CUDA events around its three kernels on `cs`, waits for them, and stores the elapsed
 * milliseconds in kernel_ms (HOST float[3]: statistics pass, table pass, encode pass).
 */
int lc_compress_timed(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                      uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs,
                      float* kernel_ms);

/*
 * Stage dumps: results of the statistics and table kernels of the last lc_compress that used
 * `workspace` (Section 3.1.1: bucket statistics; Section 3.1.2: code table). All outputs HOST. Waits for `cs`.
 *   count[512], mmin[512], mmax[512]: bucket statistics by key = 256*sign + exponent field (empty
 *   bucket: mmin 0x7FFFFF, mmax 0).
 *   len[512], code[512]: code length and canonical code of the symbol each key maps to.
 */
int lc_debug_bins(const void* workspace, uint64_t* count, uint32_t* mmin, uint32_t* mmax,
                  lc_cuda_stream_t cs);
int lc_debug_codes(const void* workspace, uint32_t* len, uint64_t* code, lc_cuda_stream_t cs);

/*
 * lc_compress with the limits of the encode pass's bounded wait exposed (the wait of the scan that places
 * the chunks, format section 3.3; the paper has no counterpart).
 *   spin_limit    polls of a predecessor's descriptor before a CTA gives up with LC_ERR_TIMEOUT
 *                 (lc_compress uses 2^20).
 *   first_ticket  number of the first tile handed out (lc_compress: 0). With 1, tile 0 is never coded, so
 *                 its descriptor never appears: the CTA that needs it gives up after spin_limit polls, its
 *                 successors see the abort mark, and every CTA returns. Nothing can hang, because every wait
 *                 is bounded; the status word then holds LC_ERR_TIMEOUT and the stream is unusable.
 */
int lc_debug_compress_wait(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                           uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, uint32_t spin_limit,
                           uint32_t first_ticket, lc_cuda_stream_t cs);

#ifdef __cplusplus
}
#endif
#endif /* LC_DEBUG_H_ */
