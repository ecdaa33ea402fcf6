/*
 * chiron_kv.h -- C ABI of the decode-iteration hot path: paged grouped-query decode attention
 * over a bf16 KV cache, and the paged KV append of each iteration's new token.
 *
 * Framing (paper): a serving instance runs a continuous batch of requests (Section 2.1,
 * "Continuous Batching"); every decode iteration generates one token per running request from
 * the keys and values of all its previous tokens, which are kept in the KV cache ("Inference
 * Primer"); the cache is managed in pages allocated on demand ("PagedAttention").  The
 * iteration's latency as a function of batch size is the quantity the local autoscaler weighs
 * against the inter-token-latency SLO (Section 4.1 "Local Backpressure", Algorithm 1).
 *
 * Conventions
 *  - All functions are extern "C", return an int32 status (CKV_OK or a negative CKV_E* code) and
 *    never throw.  ckv_last_error() gives a message for the calling thread's last failure.
 *  - "d_" pointers are DEVICE pointers, "h_" pointers are HOST pointers.  Every device buffer is
 *    owned by the caller; the library never allocates or frees device memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue
 *    work on it and return without synchronising unless stated otherwise.
 *  - bf16 values are raw 16-bit patterns (upper half of an IEEE binary32).
 *  - KV pool layout:  bf16 pool[num_layers][num_pages][num_kv_heads][2 (0=K,1=V)][page_size][head_dim]
 *    so the K and V rows of one (page, KV head) form one contiguous block.
 *  - Block tables: int32 [batch][max_pages_per_req]; entry i of row r is the physical page that
 *    holds tokens [i*page_size, (i+1)*page_size) of request r.  Only the first
 *    ceil(seq_lens[r]/page_size) entries of a row are read.  Requests may share pages for
 *    reading; append targets must be distinct.
 *  - seq_lens[r] is the context length AFTER this iteration's append: attention of request r
 *    covers tokens 0 .. seq_lens[r]-1 and the appended token has position seq_lens[r]-1.
 *  - Query head h uses KV head h / (num_q_heads / num_kv_heads).  Softmax scale is
 *    1/sqrt(head_dim).
 *  - Invalid device-side data (a length < 1 or beyond the table, a page id outside the pool) is
 *    never followed: the access is skipped or redirected to page 0, a bit is set in a device
 *    status word, and kv_check_status() reports it.  Output rows of a request with an invalid
 *    length are zero-filled; rows of a request with an invalid page id are unspecified.
 *
 * Supported shapes: head_dim 64 or 128, page_size 16, 1 <= num_q_heads/num_kv_heads <= 8.
 */
#ifndef CHIRON_KV_H
#define CHIRON_KV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CKV_OK        0
#define CKV_EINVAL   (-1)   /* bad argument or unsupported shape */
#define CKV_ENOMEM   (-2)   /* a caller-provided buffer is too small */
#define CKV_ECUDA    (-3)   /* a CUDA runtime/driver call failed (see ckv_last_error) */
#define CKV_EBOUNDS  (-4)   /* device saw an out-of-range length or page id */
#define CKV_ETIMEOUT (-5)   /* a bounded device-side wait gave up */

/* bits of the device status word */
#define CKV_STATUS_BAD_LENGTH 1u
#define CKV_STATUS_BAD_PAGE   2u
#define CKV_STATUS_WAIT_LIMIT 4u

typedef struct ckv_config {
    int32_t num_layers;         /* layers sharing block tables, each with its own pool slice */
    int32_t num_q_heads;        /* Hq */
    int32_t num_kv_heads;       /* Hkv, divides Hq */
    int32_t head_dim;           /* d: 64 or 128 */
    int32_t page_size;          /* P: 16 */
    int32_t num_pages;          /* physical pages per layer */
    int32_t max_pages_per_req;  /* row width of the block tables */
    int32_t max_batch;          /* largest batch any call will pass */
} ckv_config;

typedef struct ckv_pool ckv_pool;   /* host-side handle; holds no device allocations of its own */

/* Bytes of the KV pool for this configuration (0 if the configuration is invalid). */
size_t kv_pool_bytes(const ckv_config *cfg);

/* Bytes of scratch the library needs: status word, split-KV plan, partial results, and staging
 * for decode_step_host (0 if the configuration is invalid). */
size_t kv_workspace_bytes(const ckv_config *cfg);

/*
 * Create the host-side handle for a pool that lives in caller-owned device memory (the paged
 * KV cache of Section 2.1 "PagedAttention").  d_pool must be 256-byte aligned and hold
 * kv_pool_bytes(); d_workspace must be 256-byte aligned and hold kv_workspace_bytes().  The
 * workspace is cleared on the default stream and the call synchronises once.  `device` is the
 * CUDA device ordinal both buffers live on; the call makes it the calling thread's current
 * device and leaves it so.  Every later call that takes the handle must be made with that device
 * current and returns CKV_EINVAL otherwise (it would launch on the wrong GPU).  Errors:
 * CKV_EINVAL (shape, alignment), CKV_ENOMEM (a size too small), CKV_ECUDA.
 */
int32_t kv_pool_create(const ckv_config *cfg, void *d_pool, size_t pool_bytes,
                       void *d_workspace, size_t workspace_bytes, int32_t device,
                       ckv_pool **out_pool);

/* Free the host handle (synchronises the device first).  Device memory stays with the caller. */
int32_t kv_pool_destroy(ckv_pool *pool);

/*
 * KV append (Section 2.1 "Inference Primer": the key and value vectors of generated tokens are
 * cached for later tokens).  For each request r < batch and KV head kh, copies bit-exactly
 *   d_k_new[r][kh][:] -> pool[layer][page][kh][K][slot][:]   and   d_v_new -> ...[V]...
 * with page = d_block_tables[r][(seq_lens[r]-1)/P], slot = (seq_lens[r]-1) % P.
 * d_k_new, d_v_new: bf16 [batch][num_kv_heads][head_dim], 16-byte aligned.  No other byte of
 * the pool is written.  Errors: CKV_EINVAL (layer/batch out of range, NULL), CKV_ECUDA.
 */
int32_t kv_append(ckv_pool *pool, int32_t layer, int32_t batch,
                  const int32_t *d_block_tables, const int32_t *d_seq_lens,
                  const void *d_k_new, const void *d_v_new, void *stream);

/*
 * Decode attention for one layer of the running batch (the "self-attention computation" whose
 * cost grows with batch size, Section 2.3 "Motivation and Characterization" and Section 4.1):
 *   out[r][h][:] = sum_j softmax_j( q[r][h].k_j / sqrt(d) ) v_j ,  j over request r's context,
 * computed as split-KV partials over balanced page ranges followed by a log-sum-exp combine.
 * d_q, d_out: bf16 [batch][num_q_heads][head_dim], 16-byte aligned; every row of d_out is
 * overwritten.  Enqueues ONE kernel: the partition is derived in its prologue and partials are
 * merged by whichever warp finishes a (request, KV head) last.
 * Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t decode_attention(ckv_pool *pool, int32_t layer, int32_t batch,
                         const int32_t *d_block_tables, const int32_t *d_seq_lens,
                         const void *d_q, void *d_out, void *stream);

/*
 * One layer's whole decode iteration in ONE kernel: kv_append and decode_attention fused.  The warp
 * that processes the last tile of a (request, KV head) stores that pair's new key and value rows
 * to the pool (bit-exactly what kv_append writes) and patches them into its staged tile, so the
 * result equals kv_append followed by decode_attention (Section 2.1 "Inference Primer": each new
 * token attends to all previous tokens' keys and values, its own included, and its key/value
 * are cached).  Arguments as in those two calls.  Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t decode_step(ckv_pool *pool, int32_t layer, int32_t batch,
                    const int32_t *d_block_tables, const int32_t *d_seq_lens,
                    const void *d_q, const void *d_k_new, const void *d_v_new, void *d_out,
                    void *stream);

/*
 * Multi-token step: every request appends q_len tokens in this iteration and the q_len new tokens
 * attend causally -- new token i (position seq_lens[r] - q_len + i) sees the context up to and
 * including itself.  This is the verification pass of speculative decoding and a chunk of chunked
 * prefill, which the paper lists among the optimizations an instance may run with (Section 4,
 * "Why use an online algorithm?"; Section 6 "Experiment Setup").  seq_lens hold the lengths AFTER
 * the q_len tokens are appended; requests with seq_lens[r] < q_len are unusable (status bit, rows
 * zero-filled).
 *   kv_append_multi         d_k_new, d_v_new: bf16 [batch][q_len][num_kv_heads][head_dim]; 1 <= q_len <= 8
 *   decode_attention_multi  d_q, d_out: bf16 [batch][q_len][num_q_heads][head_dim]; 1 <= q_len <= 8.
 *                           The new tokens' queries share the 8 columns of one tensor-core pass
 *                           with the heads of the group, so while
 *                           q_len * (num_q_heads / num_kv_heads) <= 8 the KV stream is read once
 *                           for all of them.  Beyond that the step takes
 *                           ceil(q_len / (8 / group)) launches, each reading the KV stream again for
 *                           its own block of new tokens.
 * Call kv_append_multi first: attention reads the new tokens' keys and values from the pool.
 * Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t kv_append_multi(ckv_pool *pool, int32_t layer, int32_t batch, int32_t q_len,
                        const int32_t *d_block_tables, const int32_t *d_seq_lens,
                        const void *d_k_new, const void *d_v_new, void *stream);
int32_t decode_attention_multi(ckv_pool *pool, int32_t layer, int32_t batch, int32_t q_len,
                               const int32_t *d_block_tables, const int32_t *d_seq_lens,
                               const void *d_q, void *d_out, void *stream);

/*
 * The split-KV partition decode_attention uses for these lengths, copied to the host for
 * inspection (runs a small kernel and synchronises `stream`; decode_attention itself derives the
 * same partition inside its attention kernel and launches no plan kernel).  A "tile" is 32
 * consecutive tokens of one (request, KV head).  Work is laid out on an axis of units,
 * request-major then KV head: each (request, KV head) contributes CKV_PIECE_COST_TILES (3)
 * overhead units followed by one unit per tile.  Span s -- the work of one warp -- owns the tiles
 * whose units fall in [s*units_per_span, min((s+1)*units_per_span, total_units)).
 *   h_header[4]   : total_units, units_per_span, num_spans, number of spans with a non-empty range
 *   h_span_start  : int32 [num_spans][4] = request, kv head, first tile within that
 *                   (request, kv head), unit index of that tile; -1s if the span holds no tile
 * h_span_start must hold 4*ckv_get_partition() ints.  Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t decode_plan(ckv_pool *pool, int32_t batch, const int32_t *d_seq_lens, void *stream,
                    int32_t *h_header, int32_t *h_span_start);

/*
 * Read probe: streams exactly the KV tiles that decode_attention would read for this batch -- same
 * partition, same TMA boxes, same ring depth per warp -- and does nothing with them.  Its running
 * time is the practical ceiling of the memory system for this access pattern, which bench.py
 * reports beside the attention kernel ("self-attention computation" being the part of the
 * iteration that grows with the batch, Section 2.3, what bounds it is worth knowing).  Writes no
 * output; bad page ids are flagged in the status word as in decode_attention.
 * Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t kv_read_probe(ckv_pool *pool, int32_t layer, int32_t batch,
                      const int32_t *d_block_tables, const int32_t *d_seq_lens, void *stream);

/* Number of spans the partition is balanced over (default: warps per CTA x number of SMs).
 * Setting it changes only how the context is split, never the result beyond fp32 summation
 * order.  1 <= num_spans <= 2048.  Errors: CKV_EINVAL. */
int32_t ckv_set_partition(ckv_pool *pool, int32_t num_spans);
int32_t ckv_get_partition(const ckv_pool *pool);

/* Kernel overlap (default on): append and attention kernels are launched so that a kernel's
 * prologue may run under the tail of its predecessor in the stream; each waits for the
 * predecessor to complete before it first touches the pool, the workspace, q or an output.
 * The attention prologue reads d_seq_lens and d_block_tables BEFORE that wait, so with overlap on
 * they must not be produced by the kernel that immediately precedes decode_attention in the
 * stream (tables copied by a memcpy, or written by any earlier kernel, are fine -- the usual case,
 * since a serving engine uploads them once per iteration).  decode_step, being the only writer of
 * its layer's pool, also starts its first KV tile loads before that wait -- but never a tile that
 * holds position seq_lens[r]-2 or later of its (request, KV head).  Position seq_lens[r]-1 is this
 * step's own row (patched into the staged tile, whatever the copy saw); position seq_lens[r]-2 is
 * what the previous decode_step of a loop that grows every context by one token per step stored,
 * and that kernel may still be running.  Every kernel of this library releases its successor only
 * after its own wait, so the early loads overlap the immediately preceding kernel and nothing
 * older.  What follows for callers with overlap on:
 *   - a kernel of the CALLER's that immediately precedes decode_step must not write pool pages
 *     that this step reads;
 *   - if the immediately preceding kernel is a decode_step on the same layer, each request of this
 *     step must have grown by at most one token since (the same lengths replayed, as a benchmark
 *     does, are fine too); an engine that rewrites older positions in place calls kv_append or
 *     turns overlap off.
 * The library's other writers are taken care of: after kv_append, kv_append_multi or kv_swap_in
 * on this handle the next decode_step keeps all its loads behind the wait.
 * Turning overlap off restores plain stream order.  Errors: CKV_EINVAL. */
int32_t ckv_set_overlap(ckv_pool *pool, int32_t enable);

/* Synchronise `stream`, read and clear the device status word.  Returns CKV_OK, CKV_EBOUNDS
 * (bad length or page id seen), CKV_ETIMEOUT, or CKV_ECUDA.  *out_bits (may be NULL) receives
 * the raw CKV_STATUS_* bits. */
int32_t kv_check_status(ckv_pool *pool, void *stream, uint32_t *out_bits);

/*
 * Self-test of the failure path behind CKV_ETIMEOUT (test support; not part of the decode path).
 * Every wait inside the kernels is bounded: a warp that waits longer than the limit for a copy to
 * land sets CKV_STATUS_WAIT_LIMIT, stops working and returns, so a lost copy becomes an error
 * code instead of a hung GPU.  This call makes that happen on purpose and harmlessly: it enqueues
 * a one-warp kernel that waits, with the kernels' own wait routine and `limit_ns` as the limit
 * (1 us .. 100 ms), on a barrier phase that nothing completes -- no copy is issued -- and that
 * leaves arrival counter 0 raised by one, as a warp giving up inside a merge would.  Afterwards
 * kv_check_status() must report CKV_ETIMEOUT and bring the handle back to a usable state (status
 * word and arrival counters cleared).  Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t ckv_wait_limit_selftest(ckv_pool *pool, uint64_t limit_ns, void *stream);

/*
 * One whole iteration for one layer with HOST buffers: brings the tables, lengths, q, k_new and
 * v_new to the device, runs decode_step, delivers the output to h_out and synchronises `stream`.
 * Routes (ckv_set_host_route; CKV_HOST_ROUTE_AUTO picks STAGED when it applies, else COPY):
 *   CKV_HOST_ROUTE_STAGED  all six buffers are host memory the device can address (pinned or
 *                          registered, h_out 16-byte aligned): one kernel gathers the five inputs
 *                          into the workspace, the attention kernel starts under it, waits for it
 *                          before its plan and writes its output rows straight into h_out.  Two
 *                          launches, no DMA copy.
 *   CKV_HOST_ROUTE_DIRECT  same buffers (q, k_new, v_new 16-byte aligned too): the attention kernel
 *                          reads everything straight from host memory.  One launch; every read
 *                          pays the host link's latency.
 *   CKV_HOST_ROUTE_COPY    any host memory: five host-to-device copies, decode_step, one
 *                          device-to-host copy.
 * A route whose conditions are not met falls back to the next one in this order.
 * h_out: bf16 [batch][num_q_heads][head_dim].  Errors: as kv_append / decode_attention.
 */
#define CKV_HOST_ROUTE_AUTO   0
#define CKV_HOST_ROUTE_STAGED 1
#define CKV_HOST_ROUTE_DIRECT 2
#define CKV_HOST_ROUTE_COPY   3
int32_t ckv_set_host_route(ckv_pool *pool, int32_t route);
int32_t decode_step_host(ckv_pool *pool, int32_t layer, int32_t batch,
                         const int32_t *h_block_tables, const int32_t *h_seq_lens,
                         const void *h_q, const void *h_k_new, const void *h_v_new,
                         void *h_out, void *stream);

/*
 * Iteration latency against batch size: the curve Algorithm 1 reads as ITL(batch size)
 * (Section 2.1, the figure of ITL and throughput against batch size; Section 4.1).  For each
 * i < n_sizes, runs `warmup` untimed and `iters` timed
 * steps on the first batch_sizes[i] requests of the given arrays; a step is decode_step (append
 * + attention in one kernel) for every layer.  Per-layer inputs are laid out
 *   d_q, d_out [num_layers][batch_stride][Hq][d],  d_k_new, d_v_new [num_layers][batch_stride][Hkv][d].
 * Each timed step is bracketed by CUDA events on `stream`; if d_flush is not NULL, then before
 * every step (outside the timed bracket) the first half of its flush_bytes is overwritten, so
 * that no step starts with its inputs in L2, and the second half is read, so that the cache
 * holds clean lines rather than the overwrite's dirty ones, whose write-back the step would
 * otherwise pay for; give it at least twice the L2 size.  Synchronises.  out_median_us / out_min_us: [n_sizes].
 * Errors: CKV_EINVAL, CKV_ECUDA, CKV_EBOUNDS/CKV_ETIMEOUT if the status word is set afterwards.
 */
int32_t step_latency_sweep(ckv_pool *pool, int32_t n_sizes, const int32_t *batch_sizes,
                           int32_t batch_stride,
                           const int32_t *d_block_tables, const int32_t *d_seq_lens,
                           const void *d_q, const void *d_k_new, const void *d_v_new, void *d_out,
                           int32_t warmup, int32_t iters, void *d_flush, size_t flush_bytes,
                           void *stream, double *out_median_us, double *out_min_us);

/*
 * Per-kernel timing for roofline accounting: while enabled, decode_attention brackets its
 * attention kernel with CUDA events on the launch stream (up to 4096 launches are kept).
 * ckv_profile_read synchronises the device and returns the summed kernel time and the number
 * of launches since enabling.  Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t ckv_profile_enable(ckv_pool *pool, int32_t enable);
int32_t ckv_profile_read(ckv_pool *pool, double *out_attention_ms, int32_t *out_launches);

/*
 * Per-span timeline of the most recent attention kernel, for load-balance analysis (synchronises
 * `stream`).  h_trace: uint64 [ckv_get_partition()][8]: nanoseconds of the GPU's global timer at
 * warp start, first tile landed (0 if the span had no work), last tile computed, span finished;
 * then nanoseconds spent waiting for tile data, nanoseconds spent between pieces, the span's tile
 * count and its piece count.
 * h_span_start (may be NULL): int32 [ckv_get_partition()][4], the span starts the kernel derived
 * itself, in decode_plan's format.  Errors: CKV_EINVAL, CKV_ECUDA.
 */
int32_t ckv_read_span_trace(ckv_pool *pool, void *stream, uint64_t *h_trace, int32_t *h_span_start);

/* Kernels launched through this handle since creation (append, attention, plan inspection). */
int64_t ckv_launch_count(const ckv_pool *pool);

/*
 * KV swap-out / swap-in: move one request's pages, for every layer, between the pool and a
 * contiguous image in host memory (Section 3 "Request Multiplexing with Mixed Instances": an
 * interactive request may evict a batch request from a mixed instance, and the evicted request's
 * KV cache is saved by migrating it to CPU memory so that it can restart fast).
 *   d_page_ids  int32 [n_pages] on the device: the request's block-table row (physical page ids,
 *               in context order).  For swap-in these may be different pages than at swap-out.
 *   h_image     PINNED host memory (cudaHostAlloc / cudaHostRegister, 16-byte aligned) the device
 *               can address; the kernels read and write it directly, there is no staging copy.
 *               Layout: bf16 [num_layers][n_pages][num_kv_heads][2][page_size][head_dim];
 *               image_bytes >= num_layers * n_pages * (bytes of one page in one layer).
 * Both calls only enqueue one kernel on `stream`; the image is complete (swap-out) or reusable
 * (swap-in) once the stream has reached that point.  A page id outside the pool is skipped and
 * flagged in the status word.  Bit-exact.
 * Errors: CKV_EINVAL (arguments, unpinned image), CKV_ENOMEM (image too small), CKV_ECUDA.
 */
int32_t kv_swap_out(ckv_pool *pool, int32_t n_pages, const int32_t *d_page_ids, void *h_image,
                    size_t image_bytes, void *stream);
int32_t kv_swap_in(ckv_pool *pool, int32_t n_pages, const int32_t *d_page_ids, const void *h_image,
                   size_t image_bytes, void *stream);

/*
 * decode_attention without a workspace.  (The paper has no counterpart; this entry point exists
 * for integration reasons only.)
 *
 * Who it is for: code that must not, or cannot, allocate device memory at the point where it
 * needs attention -- an engine that handed all free HBM to the KV pool at start-up so that any
 * later cudaMalloc fails, a plugin running under a host framework that owns the allocator, a
 * latency-critical loop that cannot afford cudaMalloc's implicit device-wide synchronisation.
 * Such a caller has the pool, the tables and q/out, but nowhere to put the split-KV partials.
 *
 * Here they go into a fixed array inside the library's device image instead:
 * about 5.1 MiB per GPU, held by every GPU that loads the library until the process exits.  It is
 * sized for at most 640 spans (a B200 uses 592) at head_dim <= 128.  No pool handle is needed: the
 * configuration and the pool pointer are passed directly, on the CURRENT device.  The function
 * calls no cudaMalloc / cudaFree and no allocating library routine; the result is the same as
 * decode_attention's for the same partition.
 *
 *   cfg        shape of the pool (same rules as kv_pool_create; max_batch bounds `batch`)
 *   d_pool     256-byte aligned device pointer to kv_pool_bytes(cfg) bytes
 *   num_spans  partition width; 0 = warps per CTA x number of SMs.  More than 640 is rejected
 *              with CKV_EINVAL and a message -- nothing is launched.
 *   h_status   NULL: the call only enqueues work on `stream`; the device status bits of this call
 *              (bad length, bad page id, wait limit) can then not be read afterwards -- the next
 *              call clears them -- so pass NULL only for inputs known to be valid.  Otherwise the
 *              call synchronises `stream`, stores the CKV_STATUS_* bits there and returns
 *              CKV_EBOUNDS / CKV_ETIMEOUT if any is set.
 *
 * Set-up: the first call on each device looks up the array's device address
 * (cudaGetSymbolAddress), the device's SM count and the kernel's shared-memory attribute and
 * remembers them; make that first call outside any stream capture.  First calls from several
 * host threads at once are harmless (every thread would store the same values).  Later calls do
 * no look-ups: they encode the tensor map of the pool on the stack, clear the counters and launch.
 * Sharing: every call on a device uses the same array, which still holds the previous call's
 * contents; each call clears the parts that must start at zero (status word, arrival counters) on
 * `stream` before its kernel.  Two calls that can overlap on the GPU (different streams, no
 * dependency) would race on the array: keep calls on one device ordered.
 * Errors: CKV_EINVAL (shape, alignment, layer/batch range, num_spans > 640), CKV_ECUDA.
 */
int32_t decode_attention_noalloc(const ckv_config *cfg, const void *d_pool, int32_t layer, int32_t batch,
                                 const int32_t *d_block_tables, const int32_t *d_seq_lens,
                                 const void *d_q, void *d_out, int32_t num_spans, void *stream,
                                 uint32_t *h_status);

/* Message describing the calling thread's most recent failure ("" if none). */
const char *ckv_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* CHIRON_KV_H */
