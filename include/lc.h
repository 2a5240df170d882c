/*
 * lc.h - C ABI of the LC-Checkpoint compress / recover library for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-snapshot compress pass and the recovery pass of the lossy
 * delta-encoding checkpoint scheme of "On Efficient Constructions of Checkpoints" (arxiv 2009.13003):
 * Algorithm 1 steps 4-7, Section 3.1.1 (exponent-based quantization, priority promotion, midrange
 * representative) and Section 3.1.2 (Huffman coding), and the reconstruction identity
 * u_t = u_0 + sum of the quantized deltas (Section 3, after component C2).
 *
 * Conventions for every call
 *  - Pointers marked DEVICE are CUDA device pointers owned by the caller; pointers marked HOST are
 *    ordinary host pointers. The library allocates no memory. It keeps no state between calls except
 *    launch parameters that it looks up once per device (SM count, occupancy, shared-memory attributes
 *    of its kernels), and, for lc_compress_noalloc only, the built-in scratch array described there.
 *  - Work is enqueued on the CUDA stream `cs` (0 = the default stream) and, unless stated, the call
 *    returns without waiting for it. Buffers must stay valid until that work has finished.
 *  - Return value: LC_OK (0) or a negative LC_ERR_* code. Errors that only the device can see
 *    (non-finite delta, malformed stream, a bounded wait that gave up) are written to a status word
 *    in the workspace and read back with lc_last_status(). No call aborts, throws or traps.
 *  - The byte format of a stream is fixed by docs/FORMAT.md, version 1.
 */
#ifndef LC_H_
#define LC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LC_OK 0
#define LC_ERR_ARG (-1)       /* null / misaligned pointer, nbits outside 1..9, k outside 1..LC_MAX_CHAIN, n >= 2^32 */
#define LC_ERR_CAPACITY (-2)  /* stream or workspace buffer too small */
#define LC_ERR_NONFINITE (-3) /* some delta is Inf or NaN; the stream must not be used */
#define LC_ERR_FORMAT (-4)    /* malformed stream */
#define LC_ERR_MISMATCH (-5)  /* a stream's element count differs from n */
#define LC_ERR_TIMEOUT (-6)   /* a bounded device-side wait gave up */
#define LC_ERR_CUDA (-7)      /* a CUDA runtime call failed */
#define LC_ERR_RANGE (-8)     /* lc_compress_async: some |delta| >= 2, which needs the live state after it was released */

#define LC_MAX_CHAIN 8 /* most streams one lc_recover call applies */

/* Same underlying types as cudaStream_t and cudaEvent_t, so those can be passed directly. */
typedef struct CUstream_st* lc_cuda_stream_t;
typedef struct CUevent_st* lc_cuda_event_t;

/* Host copy of a stream header (format section 3.1). */
typedef struct lc_info {
  uint64_t n;              /* elements */
  uint64_t total_bytes;    /* size of the whole stream */
  uint64_t payload_bits;   /* sum of code lengths */
  uint64_t payload_offset; /* byte offset of the payload */
  uint32_t nbits;          /* bits of priority promotion */
  uint32_t nsym;           /* kept buckets + 1 */
  uint32_t max_len;        /* longest code */
  uint32_t nchunks;
  int32_t valid;           /* 1 if magic, version and constants are those of format version 1 */
  uint32_t fixed_width;    /* 1 if the stream carries fixed-width codes (format section 1.5) */
  uint32_t shard;          /* 1 if the stream is a shard's, coded with the table of a larger vector (section 1.6) */
  uint32_t cached_lengths; /* 1 if the code lengths came from a length cache (format section 1.7) */
  uint32_t mean_rep;       /* 1 if the representatives are bucket means (format section 1.8) */
} lc_info;

/* Library version (major*100 + minor). */
int lc_version(void);

/* Static text for a status code. */
const char* lc_strerror(int code);

/* Upper bound in bytes of the stream lc_compress writes for n elements (format section 6). Holds
 * because a Huffman code never uses more bits in total than the fixed nbits-bit code. */
uint64_t lc_stream_bound(uint64_t n, int nbits);

/* Bytes of DEVICE scratch lc_compress and lc_recover need for vectors of up to n elements: the control block
 * (status word, bucket statistics of Section 3.1.1, per-bucket code table), one descriptor per chunk for the
 * scan that places the chunks (format section 3.3), and one byte per element for the bucket keys that the
 * statistics pass hands to the encode pass; for lc_recover, the decode tables of the streams of one launch. */
uint64_t lc_workspace_bytes(uint64_t n);

/*
 * Compress pass (Algorithm 1 steps 4-6; Sections 3.1.1-3.1.2).
 *   stream <- LC(cur - base): the fp32 delta of `cur` against the tracked state `base` is bucketed by
 *   sign and exponent, the 2^nbits - 1 occupied buckets with the largest exponent are kept and
 *   represented by the midrange of their values, everything else becomes zero, and the bucket symbols
 *   are Huffman-coded.
 * base, cur   DEVICE, read-only, n contiguous fp32 each, 16-byte aligned.
 * n           number of elements, 0 <= n < 2^32.
 * nbits       x of the x-bit priority promotion, 1..9 (9 keeps every occupied bucket: exponent-based
 *             quantization alone, the "E" stage of Section 4.3).
 * stream      DEVICE, written; 16-byte aligned; stream_capacity >= lc_stream_bound(n, nbits).
 *             The stream's size is in its header (lc_stream_info).
 * workspace   DEVICE scratch, 256-byte aligned, workspace_bytes >= lc_workspace_bytes(n). Its contents
 *             are overwritten; two calls that overlap in time need two workspaces.
 * Host-detectable errors return at once (LC_ERR_ARG, LC_ERR_CAPACITY, LC_ERR_CUDA). A delta with
 * exponent field 255 sets LC_ERR_NONFINITE in the status word and leaves the stream without its magic.
 */
int lc_compress(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs);

/*
 * Compress pass that also advances the tracked state (Algorithm 1 steps 4-7 in one call): writes the same
 * stream as lc_compress and, in its encode pass,
 *   tracked_out_i = fl32(base_i + q_i),   q = the quantized delta the stream holds (its representative, +0 for
 *                                         the zero bucket, added like any other value),
 * which is bit for bit what lc_recover(base, {stream}) would return, without a second pass over the vector.
 * tracked_out   DEVICE, n fp32, written; 16-byte aligned. May be `base` itself (the tracked state is then updated
 *               in place: every element is read for the last time before it is written). Must not be `cur`
 *               (LC_ERR_ARG), nor overlap base or cur in any other way.
 * Everything else as for lc_compress. If the device rejects the vector (LC_ERR_NONFINITE) or a wait times out,
 * tracked_out is unspecified (with tracked_out == base: partly updated only after a time-out, untouched after
 * LC_ERR_NONFINITE).
 */
int lc_compress_update(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                       uint64_t stream_capacity, float* tracked_out, void* workspace, uint64_t workspace_bytes,
                       lc_cuda_stream_t cs);

/*
 * lc_compress / lc_compress_update with options (the same passages).
 * tracked_out   NULL for lc_compress's behaviour, else as for lc_compress_update.
 * options       0, or a combination of:
 *               LC_OPT_NO_DEVICE_WAIT: the byte offsets of the chunks (format section 3.3) come from a
 *               sizes pass and a one-CTA prefix-sum kernel instead of the decoupled look-back between running
 *               CTAs of the encode pass. No kernel of the call then ever waits for another CTA, so
 *               LC_ERR_TIMEOUT cannot occur; the price is one more pass over the one-byte key plane.
 *               For deployments where a device-side spin, however bounded, is not acceptable.
 *               LC_OPT_FIXED_WIDTH: the bucket indices are written with ceil(log2 nsym) bits each instead of their
 *               Huffman codes (format section 1.5): the stream of Section 3.1.1's size model, n*ceil(log2 k) bits
 *               of indices, and the "E" (with nbits 9) and "E+P" stages of Section 4.3's size breakdown as real
 *               streams. lc_recover reads such streams like any other. This option does change the bytes.
 *               LC_OPT_MEAN_REP: a bucket is represented by the mean of its values, rounded once to fp32, instead
 *               of the average of its maximum and minimum that Section 3.1.1 prescribes (format section 1.8). A
 *               variant, not the paper's method: the mean minimises the squared error inside a bucket. Symbols,
 *               code and payload are unchanged; only the table's representatives (and so the recovered values)
 *               differ. The statistics pass then also sums the mantissas, exactly and in integers, so the result
 *               is as deterministic as the default; that pass runs about 1.35 times as long. Not together with
 *               LC_OPT_FIXED_WIDTH (LC_ERR_ARG).
 * Any other bit in `options` returns LC_ERR_ARG.
 */
#define LC_OPT_NO_DEVICE_WAIT 1u
#define LC_OPT_FIXED_WIDTH 2u
#define LC_OPT_MEAN_REP 4u
int lc_compress_opt(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                    uint64_t stream_capacity, float* tracked_out, void* workspace, uint64_t workspace_bytes,
                    uint32_t options, lc_cuda_stream_t cs);

/*
 * Per-layer granularity. The paper compresses "the model state"; whether layer by layer or as one vector it does not
 * say. These calls cut the vector into nseg contiguous segments (the layers of a model) and code every segment as a
 * complete stream of its own, with its own buckets, representatives and code (Sections 3.1.1 and 3.1.2 applied per
 * segment): layers whose updates differ in scale then each keep their own top 2^nbits - 1 buckets. Each segment's
 * stream is byte for byte what lc_compress writes for that slice of base and cur.
 * seg_begin     HOST, nseg + 1 element offsets, seg_begin[0] = 0, non-decreasing, every one a multiple of 4 (the
 *               segments then start on 16-byte boundaries), each segment shorter than 2^32 elements;
 *               1 <= nseg <= LC_MAX_SEGMENTS. The vector has seg_begin[nseg] elements.
 * lc_segments_layout: where the streams go. Segment i's stream starts at byte stream_offset[i] of the streams buffer
 *               (its slot ends at stream_offset[i + 1]: lc_stream_bound of the segment, rounded up to 256);
 *               stream_offset (HOST, nseg + 1 entries) may be NULL. Returns the buffer size needed, 0 on bad arguments.
 * streams       DEVICE, 256-byte aligned, streams_capacity >= lc_segments_layout(...). For lc_recover_segments: HOST
 *               array of k such buffers, applied in array order (1 <= k <= LC_MAX_CHAIN).
 * tracked_out   NULL, or as for lc_compress_update (the whole vector; may be base).
 * workspace     as for lc_compress, of lc_workspace_bytes(longest segment) bytes; one status word for the call: the
 *               first failure of any segment stays in it (lc_last_status), and the segments after a failed one are
 *               left without a valid stream (compress) or with unspecified output (recover).
 * The segments run one after the other on `cs`, a handful of launches each: this is for models of tens to hundreds
 * of layers, not for millions of tiny tensors.
 */
#define LC_MAX_SEGMENTS 65536
uint64_t lc_segments_layout(const uint64_t* seg_begin, int nseg, int nbits, uint64_t* stream_offset);
int lc_compress_segments(const float* base, const float* cur, const uint64_t* seg_begin, int nseg, int nbits,
                         void* streams, uint64_t streams_capacity, float* tracked_out, void* workspace,
                         uint64_t workspace_bytes, lc_cuda_stream_t cs);
int lc_recover_segments(const float* base, const void* const* streams, int k, const uint64_t* seg_begin, int nseg,
                        int nbits, float* out, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs);

/*
 * lc_compress / lc_compress_update with the code table of an earlier snapshot (Section 3.2, "Huffman Code Table
 * Caching": when the number of buckets is the same as before, the table is used again, the buckets only being
 * sorted by their numbers of entries). The cache is the caller's: LC_LENGTH_CACHE_BYTES of DEVICE memory, 16-byte
 * aligned, all zero before its first use, passed to every call that should share it; the calls that share one
 * cache must be ordered (same CUDA stream, or events). Format section 1.7 defines its rows and the rule: with u
 * used symbols, a valid row u - 1 gives the r-th most frequent symbol the row's r-th length, provided the payload
 * then stays within n * nbits bits; otherwise the Huffman lengths are built as usual and stored in the row.
 * A stream coded with cached lengths has `cached_lengths` set in its lc_info, is read by lc_recover like any other,
 * and recovers exactly the state the plain stream recovers; only its size may be larger, since the code is the
 * optimal one of another snapshot. On this hardware the table pass is about 1 % of the call, so the cache saves
 * next to nothing here: it is provided because the paper's system has it.
 * tracked_out   NULL for lc_compress's behaviour, else as for lc_compress_update.
 * length_cache  NULL or misaligned returns LC_ERR_ARG.
 */
#define LC_LENGTH_CACHE_BYTES 262144u
int lc_compress_cached(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                       uint64_t stream_capacity, float* tracked_out, void* workspace, uint64_t workspace_bytes,
                       void* length_cache, lc_cuda_stream_t cs);

/*
 * Recovery pass (Algorithm 1 step 7 applied k times; u_t = u_0 + sum_i quantized delta_i).
 *   out_i = fl32(...fl32(fl32(base_i + d_0,i) + d_1,i)... + d_{k-1},i), streams applied in array order.
 * base          DEVICE, n fp32, 16-byte aligned.
 * streams       HOST array of k DEVICE pointers (16-byte aligned) to streams written by lc_compress.
 * stream_bytes  HOST array of k buffer sizes in bytes; no byte beyond them is read.
 * k             1..LC_MAX_CHAIN.
 * n             elements in base and out; every stream's header must say the same n.
 * out           DEVICE, n fp32, 16-byte aligned; may be the same pointer as base (in-place update).
 * workspace     as for lc_compress; lc_workspace_bytes(0) is enough for any n (the status word and the decode
 *               tables of the streams live there).
 * Malformed streams set LC_ERR_FORMAT / LC_ERR_MISMATCH in the status word; `out` is then unspecified
 * but no out-of-bounds access happens.
 */
int lc_recover(const float* base, const void* const* streams, const uint64_t* stream_bytes, int k,
               uint64_t n, float* out, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs);

/*
 * Compress pass split over two CUDA streams (Section 3.2, "Asynchronous Execution": only the first step of the
 * checkpointing process, the delta against the live model state, depends on that state; the rest can run beside
 * the next training iteration).
 * The statistics pass, the only one that reads base and cur, is enqueued on `cs_state` (the stream that owns the
 * model state), followed by a record of `state_read` on that stream. The table and encode passes are enqueued on
 * `cs_side` behind a wait for that event. Work enqueued on cs_state after this call therefore waits for the
 * statistics pass only, and may overwrite cur (and base) as soon as it runs; the stream is complete when cs_side
 * has drained.
 *   state_read  an event created by the caller (cudaEventCreateWithFlags(..., cudaEventDisableTiming) is enough);
 *               recorded by this call. cs_state and cs_side must be different streams of one device.
 * Everything else as for lc_compress, with one restriction: the statistics pass hands the encode pass one byte
 * per element, which identifies the bucket only while every |delta| < 2 (exponent field below 128). lc_compress
 * falls back to reading base and cur again in that case; this call cannot, because it has released them, and
 * reports LC_ERR_RANGE in the status word instead (the stream is then unusable; use lc_compress).
 */
int lc_compress_async(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                      uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs_state,
                      lc_cuda_stream_t cs_side, lc_cuda_event_t state_read);

/*
 * A vector split over several devices (each holds a contiguous shard of the model state, as under sharded data
 * parallelism). The method's table, i.e. which buckets priority promotion keeps, their representatives and the
 * Huffman code (Sections 3.1.1-3.1.2), is a function of the 512 bucket statistics of the WHOLE vector; everything
 * else is local to a shard. So the pass splits in two around one small exchange:
 *   1. lc_shard_stats on every shard: the statistics pass; the shard's statistics are left in `stats`.
 *   2. the caller combines the shards' `stats` buffers, element-wise: bytes [0, 4096) are 512 counts (u64): add;
 *      bytes [4096, 8192) are 1024 u32 words (running maxima that stand for the buckets' minima and maxima): take
 *      the maximum, as unsigned numbers. (An all-reduce of 8 KB; every shard must end up with the combined buffer.)
 *   3. lc_shard_encode on every shard, with the combined statistics: table pass and encode pass. All shards derive
 *      the same table; each writes a complete stream of its own elements, marked as a shard's (format section 1.6:
 *      its table lists the shard's own counts, and may give codes to symbols the shard does not use).
 * lc_recover applies a shard's stream to the shard's part of the base like any other stream; part by part the result
 * is what the stream of the whole vector would recover, bit for bit.
 * base, cur, n, nbits, stream, stream_capacity, workspace: as for lc_compress, for the shard; the same workspace in
 * both calls (the second uses what the first left there). stats / whole_stats: DEVICE, LC_STATS_BYTES, 16-byte aligned.
 */
#define LC_STATS_BYTES 8192
int lc_shard_stats(const float* base, const float* cur, uint64_t n, void* stats, void* workspace,
                   uint64_t workspace_bytes, lc_cuda_stream_t cs);
int lc_shard_encode(const float* base, const float* cur, uint64_t n, int nbits, const void* whole_stats, void* stream,
                    uint64_t stream_capacity, void* workspace, uint64_t workspace_bytes, lc_cuda_stream_t cs);

/*
 * Checkpoint merging (Section 3.2, "Checkpoint Merging"): the k streams that lead from `base` to a later tracked
 * state become one super-step stream, so that a later recovery applies one stream instead of k.
 * The paper does not say how the merged checkpoint is coded. The reading taken here is the scheme applied once more
 * to the summed change:
 *   merged <- LC(recover(base, streams) - base),
 * i.e. lc_recover followed by lc_compress against the same base, in one call. The merged stream quantizes a second
 * time: recovering it gives a state within the quantization error of, not bit-identical to, the state the k streams
 * recover (their sum takes many more distinct values than one stream's buckets have representatives).
 * base, streams, stream_bytes, k, n   as for lc_recover.
 * nbits, stream, stream_capacity      as for lc_compress: the merged stream.
 * scratch    DEVICE, n fp32, 16-byte aligned, written: receives recover(base, streams), which is also the state the
 *            merged stream was coded from. Must not overlap base or the streams.
 * workspace  as for lc_compress.
 * Errors as for lc_recover and lc_compress (malformed input stream, non-finite merged delta, buffers too small).
 */
int lc_merge(const float* base, const void* const* streams, const uint64_t* stream_bytes, int k, uint64_t n,
             int nbits, void* stream, uint64_t stream_capacity, float* scratch, void* workspace,
             uint64_t workspace_bytes, lc_cuda_stream_t cs);

/* Copies a stream's header to the host. `stream` DEVICE, `info` HOST. Waits for `cs`. */
int lc_stream_info(const void* stream, lc_info* info, lc_cuda_stream_t cs);

/* Waits for `cs`, then returns the status word of the last call that used `workspace`. */
int lc_last_status(const void* workspace, lc_cuda_stream_t cs);

/*
 * Host-buffer variants: the same two passes (Algorithm 1 steps 4-6 and step 7) for callers whose state lives
 * in host memory (pinned memory makes the copies asynchronous). Every transfer is part of the call: base,
 * cur -> device, stream -> host for compress; base, streams -> device, out -> host for recover. The device
 * memory comes from `arena` (DEVICE, 256-byte aligned, arena_bytes >= lc_host_arena_bytes()); the calls wait
 * for `cs` before returning and return the device status as well.
 * lc_host_arena_bytes: the workspace plus device copies of everything a call moves (two vectors and a
 * worst-case stream for compress; one vector and k worst-case streams for recover), whichever is larger.
 */
uint64_t lc_host_arena_bytes(uint64_t n, int nbits, int k);

/* base_host, cur_host HOST fp32[n]; stream_host HOST, capacity >= lc_stream_bound; *stream_bytes_out
 * receives the stream size. */
int lc_compress_host(const float* base_host, const float* cur_host, uint64_t n, int nbits,
                     void* stream_host, uint64_t stream_capacity, uint64_t* stream_bytes_out,
                     void* arena, uint64_t arena_bytes, lc_cuda_stream_t cs);

/* base_host HOST fp32[n]; streams_host HOST array of k HOST pointers; out_host HOST fp32[n]. A vector of 128
 * chunks or more goes through in eight slices of whole chunks: slice i of base arrives on a copy stream the call
 * creates, is recovered in place on `cs`, and leaves on a second copy stream while slice i + 1 arrives, so that
 * with pinned buffers the two directions of the host link are busy at once. Both streams and their events are
 * destroyed before the call returns. */
int lc_recover_host(const float* base_host, const void* const* streams_host,
                    const uint64_t* stream_bytes, int k, uint64_t n, float* out_host, void* arena,
                    uint64_t arena_bytes, lc_cuda_stream_t cs);

/*
 * Compress pass without a caller-supplied workspace. (No counterpart in the paper: this is a
 * deployment variant of lc_compress.)
 *
 * For callers that must not allocate device memory when they take a snapshot: a trainer whose
 * memory pool already owns the whole device, code inside a region where cudaMalloc is forbidden or
 * would stall the device, a plug-in that is handed raw pointers only. The scratch memory that
 * lc_compress takes from its caller is here a fixed array inside the library image, so the call
 * allocates nothing (no cudaMalloc, cudaFree or allocating library routine) and serves vectors of at
 * most LC_NOALLOC_MAX_N elements; a larger n returns LC_ERR_CAPACITY.
 *
 *  - base, cur, n, nbits, stream, stream_capacity: exactly as for lc_compress (DEVICE pointers,
 *    16-byte aligned); the stream written is byte-identical to lc_compress's.
 *  - The call waits for `cs` and returns the device status as well (LC_ERR_NONFINITE, LC_ERR_TIMEOUT).
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current). With CUDA's default lazy module loading that look-up is also what loads the
 *    part of the library that holds the array, i.e. the moment the driver reserves the array's device
 *    memory, and it may synchronise the device. A caller whose pool is about to take the whole device
 *    must therefore make that first call at start-up, before the pool grows (n = 0 is enough: it does
 *    the look-up and writes a header-only stream), or run with CUDA_MODULE_LOADING=EAGER. Make it
 *    outside any CUDA stream capture. Later calls allocate nothing.
 *  - Every call on a device shares the one array, which keeps the previous call's contents (the call
 *    clears what must start at zero). Two calls that overlap on the same GPU race: do not issue them
 *    from different streams or threads at the same time.
 *  - The array (about 4.3 MB) stays resident on every GPU that loads the library, until exit.
 */
#define LC_NOALLOC_MAX_N 4194304ull
int lc_compress_noalloc(const float* base, const float* cur, uint64_t n, int nbits, void* stream,
                        uint64_t stream_capacity, lc_cuda_stream_t cs);

#ifdef __cplusplus
}
#endif
#endif /* LC_H_ */
