// Device code of the decode-iteration hot path for sm_100a: KV append, split-KV plan,
// paged grouped-query partial attention (TMA-fed, tensor-core) with its log-sum-exp combine.
//
// Pool layout (bf16): [layer][page][kv_head][K|V][slot 0..15][d]  -- one (page, kv_head) is a
// contiguous block of 32 rows (16 key rows, then 16 value rows) of d elements.
#pragma once

#include <cuda.h>            // CUtensorMap (type only; the driver library is not linked)
#include <cuda_runtime.h>
#include <stdint.h>

namespace ckv {

constexpr int kPageSize = 16;        // tokens per page
#ifndef CKV_PAGES_PER_TILE
#define CKV_PAGES_PER_TILE 2
#endif
constexpr int kPagesPerTile = CKV_PAGES_PER_TILE;   // a tile is the scheduling unit: 32 tokens of one (request, kv head)
constexpr int kTileTokens = kPageSize * kPagesPerTile;
constexpr int kMaxGroup = 8;         // query heads per KV head handled by one MMA column block
constexpr int kMaxSpans = 2048;      // upper bound on the partition width (one span per warp)
constexpr int kMaxBatch = 8192;
constexpr int kTreeFrom = 24;        // pairs cut into more partials than this are merged in two levels

constexpr uint32_t kStatusBadLength = 1u;
constexpr uint32_t kStatusBadPage = 2u;
constexpr uint32_t kStatusWaitLimit = 4u;

constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // bound of every device-side wait

// The split-KV partition.  Work is laid out on one axis of "units", request-major, then kv head:
// every (request, kv head) contributes kPieceCostTiles overhead units (the fixed cost of starting,
// finishing and merging a piece: three tiles' worth of time balanced best across the workloads) followed by one unit
// per tile.  Span s owns the tiles whose units fall in [s*q, min((s+1)*q, total)), q =
// ceil(total/spans), so spans that hold many short (request, kv head) pieces get fewer tiles.
#ifndef CKV_PIECE_COST_TILES
#define CKV_PIECE_COST_TILES 3
#endif
constexpr int kPieceCostTiles = CKV_PIECE_COST_TILES;

// Partials per first-level group of a two-level merge of n partials: a power of two near sqrt(n).
__host__ __device__ __forceinline__ int merge_group_size(int n)
{
    int sub = 8;
    while (sub * sub < n) sub *= 2;
    return sub;
}

struct PlanHeader {
    int32_t total_units;
    int32_t units_per_span;
    int32_t num_spans;
    int32_t spans_with_units;
};

// A context length is usable if min_len <= L <= table capacity (min_len = the number of new
// tokens of the step, 1 for plain decode); otherwise the request has no tiles.
__host__ __device__ __forceinline__ int tiles_of_length(int L, int max_pages_per_req, int min_len = 1)
{
    if (L < min_len || (long long)L > (long long)max_pages_per_req * kPageSize) return 0;
    return (L + kTileTokens - 1) / kTileTokens;
}

// ------------------------------------------------------------------------------------------
// K1: KV append.  One thread moves one 16-byte piece of one new key or value row.
// ------------------------------------------------------------------------------------------
struct AppendParams {
    uint4 *pool_layer;              // base of this layer's pool slice
    const int32_t *block_tables;
    const int32_t *seq_lens;
    const uint4 *k_new;
    const uint4 *v_new;
    uint32_t *status;
    int32_t batch, max_pages_per_req, num_pages, num_kv_heads, head_dim;
    int32_t q_len;                  // new tokens per request: k_new, v_new are [batch][q_len][Hkv][d]
};

__global__ void kv_append_kernel(const AppendParams p)
{
    // The pool may still be read by the attention kernel launched before this one: wait for the
    // predecessor before the first write, then let the next kernel start its prologue.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int vec_per_row = p.head_dim / 8;                       // 16-byte pieces per row
    const int per_tok = p.num_kv_heads * 2 * vec_per_row;
    const int per_req = per_tok * p.q_len;
    const long long total = (long long)p.batch * per_req;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(idx / per_req);
        int rem = (int)(idx % per_req);
        const int qi = rem / per_tok;                                 // which of the request's new tokens
        rem -= qi * per_tok;
        const int kh = rem / (2 * vec_per_row);
        rem -= kh * 2 * vec_per_row;
        const int kv = rem / vec_per_row;
        const int c = rem % vec_per_row;

        const int L = p.seq_lens[r];
        if (tiles_of_length(L, p.max_pages_per_req, p.q_len) == 0) {
            if (rem == 0 && kh == 0) atomicOr(p.status, kStatusBadLength);
            continue;
        }
        const int pos = L - p.q_len + qi;
        const int page = p.block_tables[(size_t)r * p.max_pages_per_req + pos / kPageSize];
        if (page < 0 || page >= p.num_pages) {
            if (rem == 0 && kh == 0) atomicOr(p.status, kStatusBadPage);
            continue;
        }
        const int slot = pos % kPageSize;
        const uint4 *src = (kv == 0 ? p.k_new : p.v_new) + (((size_t)r * p.q_len + qi) * p.num_kv_heads + kh) * vec_per_row + c;
        const size_t row = (((size_t)page * p.num_kv_heads + kh) * 2 + kv) * kPageSize + slot;
        p.pool_layer[row * vec_per_row + c] = *src;
    }
}

// ------------------------------------------------------------------------------------------
// KV swap: one request's pages, all layers, between the pool and a contiguous image in pinned host
// memory that the device reaches directly (no staging copy).  One thread moves 16 bytes at a time.
// Image layout: [layer][i][kv_head][K|V][slot][d], i = position in page_ids.
// ------------------------------------------------------------------------------------------
struct SwapParams {
    uint4 *pool;                    // whole pool
    uint4 *image;                   // device-visible address of the host image
    const int32_t *page_ids;        // [n_pages]
    uint32_t *status;
    int32_t n_pages, num_layers, num_pages;
    int32_t page_vecs;              // 16-byte pieces per (layer, page): Hkv*2*16*d*2/16
};

template <bool kToHost>
__global__ void kv_swap_kernel(const SwapParams p)
{
    const long long per_layer = (long long)p.n_pages * p.page_vecs;
    const long long total = per_layer * p.num_layers;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int layer = (int)(idx / per_layer);
        const long long rem = idx % per_layer;
        const int i = (int)(rem / p.page_vecs), v = (int)(rem % p.page_vecs);
        const int page = __ldg(p.page_ids + i);
        if (page < 0 || page >= p.num_pages) {
            if (v == 0 && layer == 0) atomicOr(p.status, kStatusBadPage);
            continue;
        }
        uint4 *in_pool = p.pool + ((size_t)layer * p.num_pages + page) * p.page_vecs + v;
        if (kToHost) p.image[idx] = *in_pool;
        else *in_pool = p.image[idx];
    }
}

// ------------------------------------------------------------------------------------------
// Gather of one step's inputs from pinned host memory that the device addresses directly: up to
// five arrays (tables, lengths, q, new keys, new values) move to their device staging areas in one
// launch instead of one DMA copy each.  Sizes are multiples of 4 bytes.
// ------------------------------------------------------------------------------------------
struct GatherParams {
    const uint8_t *src[5];
    uint8_t *dst[5];
    unsigned long long bytes[5];
};

__global__ void host_gather_kernel(const GatherParams p)
{
    // the attention kernel that follows may become resident right away; it waits for this grid
    // before it reads anything
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t tid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, nthr = (size_t)gridDim.x * blockDim.x;
#pragma unroll
    for (int a = 0; a < 5; ++a) {
        const uint8_t *src = p.src[a];
        uint8_t *dst = p.dst[a];
        const size_t bytes = p.bytes[a];
        const bool vec = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) == 0;
        const size_t nvec = vec ? bytes / 16 : 0;
        for (size_t i = tid; i < nvec; i += nthr)
            reinterpret_cast<uint4 *>(dst)[i] = reinterpret_cast<const uint4 *>(src)[i];
        for (size_t i = nvec * 4 + tid; i < bytes / 4; i += nthr)
            reinterpret_cast<uint32_t *>(dst)[i] = reinterpret_cast<const uint32_t *>(src)[i];
    }
}

// ------------------------------------------------------------------------------------------
// Cache flush helper of the latency sweep: read `vecs` 16-byte pieces once.  Run after a buffer
// larger than the L2 has been overwritten, it replaces the dirty lines that the overwrite left
// in the cache by clean ones, so the step timed next does not pay for their write-back.
// ------------------------------------------------------------------------------------------
__global__ void l2_read_sweep_kernel(const uint4 *__restrict__ src, size_t vecs, uint32_t *sink)
{
    uint32_t acc = 0;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < vecs; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = src[i];
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    if (acc == 0x9e3779b9u && sink) *sink = acc;         // keeps the loads alive; practically never taken
}

// ------------------------------------------------------------------------------------------
// K2: the split-KV plan.
//
// The attention kernel derives its partition from seq_lens in its own prologue (warp_plan below),
// so a decode step launches no separate plan kernel.  splitkv_plan_kernel computes the same
// partition for every span at once, for inspection through decode_plan().
// ------------------------------------------------------------------------------------------
struct SpanStart {
    int r, h, tile;        // first tile of the span: request, kv head, tile within (r, h); r = -1: no tile
    int tiles_r;           // tiles per kv head of request r
    int L;                 // context length of request r
    long long v;           // unit index of that first tile
    long long end;         // one past the span's last unit
    int total, q;          // header values
};

// Requests with an unusable length get their output rows cleared and the status word flagged.
// Executed by one warp of the grid.
__device__ __forceinline__ void flag_unusable_requests(const int32_t *__restrict__ seq_lens, int batch,
                                                       int max_pages_per_req, int min_len, int lane, uint16_t *out,
                                                       int out_row_elems, uint32_t *status)
{
    for (int base = 0; base < batch; base += 32) {
        const int r = base + lane;
        const bool bad = r < batch && tiles_of_length(__ldg(seq_lens + r), max_pages_per_req, min_len) == 0;
        unsigned todo = __ballot_sync(0xffffffffu, bad);
        if (todo && lane == 0) atomicOr(status, kStatusBadLength);
        while (todo) {                                   // the whole warp clears one row at a time
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            uint16_t *row = out + (size_t)(base + src) * out_row_elems;
            for (int i = lane; i < out_row_elems; i += 32) row[i] = 0;
        }
    }
}

// Units of one kv head of a request with t tiles (0 if the request is unusable).
__device__ __forceinline__ int units_of_tiles(int t) { return t > 0 ? t + kPieceCostTiles : 0; }

// Executed by one whole warp.  Two passes over seq_lens: the total number of units, then the
// (request, kv head) that holds unit span*q and the first tile at or after it.
__device__ __forceinline__ SpanStart warp_plan(const int32_t *__restrict__ seq_lens, int batch, int max_pages_per_req,
                                               int num_kv_heads, int num_spans, int span, int lane, int min_len = 1)
{
    SpanStart s;
    int sum = 0;
    for (int base = 0; base < batch; base += 32) {
        const int r = base + lane;
        if (r < batch) sum += units_of_tiles(tiles_of_length(__ldg(seq_lens + r), max_pages_per_req, min_len));
    }
#pragma unroll
    for (int x = 16; x > 0; x >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, x);
    s.total = sum * num_kv_heads;
    s.q = max(1, (s.total + num_spans - 1) / num_spans);
    const long long begin = (long long)span * s.q;
    s.r = -1; s.h = s.tile = s.tiles_r = s.L = 0;
    s.v = s.end = min(begin, (long long)s.total);
    if (begin >= s.total) return s;
    s.end = min(begin + s.q, (long long)s.total);

    long long running = 0;                               // units (all heads) before request `base`
    for (int base = 0; base < batch; base += 32) {
        const int r = base + lane;
        const int L = r < batch ? __ldg(seq_lens + r) : 0;
        const int t = r < batch ? tiles_of_length(L, max_pages_per_req, min_len) : 0;
        int incl = units_of_tiles(t);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const long long upto = running + (long long)incl * num_kv_heads;     // units through request r
        const unsigned hit = __ballot_sync(0xffffffffu, upto > begin);
        if (hit) {
            const int src = __ffs(hit) - 1;
            const int t_r = __shfl_sync(0xffffffffu, t, src);
            const int L_r = __shfl_sync(0xffffffffu, L, src);
            const int u_r = t_r + kPieceCostTiles;
            const long long before = __shfl_sync(0xffffffffu, upto, src) - (long long)u_r * num_kv_heads;
            const int rem = (int)(begin - before);
            const int h = rem / u_r, off = rem % u_r;
            const int tile = max(0, off - kPieceCostTiles);               // a span starting in the overhead
            const long long v = before + (long long)h * u_r + kPieceCostTiles + tile;   // units starts at tile 0
            if (v >= s.end) return s;                                      // the span holds overhead units only
            s.r = base + src; s.tiles_r = t_r; s.L = L_r;
            s.h = h; s.tile = tile; s.v = v;
            return s;
        }
        running = __shfl_sync(0xffffffffu, upto, 31);
    }
    return s;                                            // not reached: begin < total
}

struct PlanParams {
    const int32_t *seq_lens;
    PlanHeader *header;
    int4 *span_start;               // [num_spans] request, kv head, tile, unit index of that tile (-1s if idle)
    int32_t batch, max_pages_per_req, num_kv_heads, num_spans;
};

__global__ void splitkv_plan_kernel(const PlanParams p)
{
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int span = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; span < p.num_spans; span += warps) {
        const SpanStart s = warp_plan(p.seq_lens, p.batch, p.max_pages_per_req, p.num_kv_heads, p.num_spans, span, lane);
        if (lane == 0) {
            p.span_start[span] = s.r < 0 ? make_int4(-1, -1, -1, -1) : make_int4(s.r, s.h, s.tile, (int)s.v);
            if (span == 0) {
                p.header->total_units = s.total;
                p.header->units_per_span = s.q;
                p.header->num_spans = p.num_spans;
                p.header->spans_with_units = (s.total + s.q - 1) / s.q;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *ptr)
{
    return (uint32_t)__cvta_generic_to_shared(ptr);
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done;
}

// Wait for a phase of an mbarrier, giving up after kWaitLimitNs.  Returns false when it gave up;
// the status word is flagged and the caller stops working.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t *status,
                                                  unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) {
            atomicOr(status, kStatusWaitLimit);
            return false;
        }
    }
}

// L2 policy for data that is read once: such lines are the first to be evicted, so the stream of KV
// tiles does not push tables, queries and partial results out of the cache.
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may
// start while its predecessor in the stream still runs.  grid_dependency_wait() blocks until the
// predecessor has completed and its writes are visible; without the attribute it returns at once.
// Start fetching a tensor map (a kernel parameter) so that the first tile load does not wait for it.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void grid_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier (16-byte aligned, size % 16 == 0)
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ float4 ld_shared_f32x4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float ld_cg_f32(const float *p)
{
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ float4 ld_cg_f32x4(const float *p)
{
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// ------------------------------------------------------------------------------------------
// K3 + K4: paged partial attention with the log-sum-exp combine folded in.
//
// Every WARP is an independent worker: it owns one span of the plan, a private ring of NS stages
// in shared memory with one mbarrier per stage, a small staging tile and a parking buffer.  A stage
// holds one tile (2 pages: 32 key rows and 32 value rows of one kv head).  The warp itself issues
// the TMA box loads of the tile NS stages ahead of the one it computes on (an "issue" cursor and a
// "compute" cursor walk the same span), so there is no producer warp and, after one barrier at the
// kernel's start, no CTA-wide synchronisation; a CTA is W such warps sharing an SM's shared memory.
//
// MMA formulation (operands swapped so the tile's tokens fill the M dimension):
//   S^T[tok 16 x g 8]  = K[tok 16 x d] . Q^T[d x g 8]          (A = K rows via ldmatrix)
//   O^T[d 16 x g 8]   += V^T[d 16 x tok 16] . P^T[tok 16 x g 8] (A = V via ldmatrix.trans)
// The S^T accumulator fragment holds (token = lane/4 [+8], g = 2*(lane%4)+{0,1}); packed to bf16
// and transposed with movmatrix it is exactly the B fragment of P^T.
//
// Fused append (k_new != NULL): the warp whose span holds the LAST tile of a (request, kv head)
// owns that pair's append.  It stores the new key and value rows to the pool for later
// iterations, and overwrites the same rows of its staged tile in shared memory before computing
// on it -- so this iteration sees the new token whether the tile's copy read the pool before or
// after the store landed.  No other warp reads that slot as a live token in this launch.
//
// A piece is the part of one (request, kv head) that falls inside the span.  When it covers the
// whole context the warp normalises and writes the bf16 output rows itself.  Otherwise its fp32
// partial (m, l, O) waits in shared memory until the span has been streamed and is then merged in
// two stages, both wait-free (nobody ever waits for another warp; whoever arrives last does the
// work): the warps of a CTA that hold pieces of one (request, kv head) count themselves in on a
// shared-memory counter and the last one folds their partials; if the pair continues in other CTAs
// the folded result goes to global memory as the CTA's one partial of it, an arrival counter in
// global memory is bumped, and the last CTA to arrive merges the CTAs' partials.
// ------------------------------------------------------------------------------------------
struct AttnParams {
    const int32_t *block_tables;
    const int32_t *seq_lens;
    const uint16_t *q;
    uint16_t *out;
    // fused KV append (all three NULL for attention alone): the new token's rows and this layer's pool slice
    const uint4 *k_new;             // bf16 [batch][Hkv][d]
    const uint4 *v_new;
    uint4 *pool_layer;
    float *part;                    // [2*kMaxSpans][16 + 8*D]: a partial is (m[8], l[8]), then its rows [8][D];
                                    //   two slots per CTA are used: 2*cta, 2*cta + 1
    int32_t *arrivals;              // [kMaxSpans], all zero between launches
    int4 *span_start;               // [kMaxSpans] what each span started at (diagnostic)
    unsigned long long *trace;      // [kMaxSpans][8] ns: start, first tile landed, last tile done, span done,
                                    //   total wait for data, total time between pieces, tiles, pieces
    uint32_t *status;
    int32_t batch, max_pages_per_req, num_pages, num_kv_heads, num_q_heads, group;
    int32_t layer_page_base;        // layer * num_pages
    int32_t num_spans;
    int32_t q_len;                  // new tokens per request in this step (1 for plain decode)
    int32_t early_loads;            // > 0: the first tile loads may be issued before the dependency wait (fused step only);
                                    // < 0: even seq_lens and the tables come from the preceding kernel: wait before the plan
    int32_t q_base, q_pass;         // this launch computes new tokens q_base .. q_base + q_pass - 1; q_pass*group <= 8
    float scale_log2;               // log2(e) / sqrt(d)
};

// Columns.  The 8 columns of the MMA hold (new token, head of the group) pairs: column c is new
// token q_base + c / G and head c % G, ncols = q_pass * G <= 8 of them are live.  A step with more
// new tokens than fit is run as several launches, each over the whole KV stream with its own
// q_base.  With one new token per request (the usual decode step) a column is simply a head.
// Output rows of a (request, kv head) start at out_rows (new token q_base); column c's row is
// out_rows + (c / G) * qi_stride + (c % G) * D.
//
// ---- the fold: ONE routine merges partials, wherever they come from ------------------------
//
// A partial is the triple (m, l, O) of a (request, kv head) over part of its context: m[8] the
// reference the exponentials were taken against (log2 domain), l[8] their sums, O[8][D] the
// weighted value sums, one row per column.  In memory it is `rows` (ncp rows of D floats at some
// pitch) plus 16 floats (m[8], l[8]).  ncp is the live column count rounded up to a power of two
// (at least 128 / D), so that the ncp * D floats of the rows split evenly over the 32 lanes: the
// 32 / ncp lanes of ONE row g take its float4 pieces in turn (lane r of the row owns pieces r,
// r + 32 / ncp, ...: J = ncp * D / 128 of them), which keeps shared-memory reads conflict-free
// and global stores coalesced.  A lane therefore needs one factor per partial, not eight, and the code below has
// no per-column unrolling: it is small, which matters because every warp runs it once, after its
// span, from an instruction cache that has held nothing but the streaming loop.
//
// Folding n partials in a fixed order t = 0 .. n-1:  M = max m_t, f_t = 2^(m_t - M),
// L = sum f_t l_t, O = sum f_t O_t, in rounds of at most `cap` partials with the running (M, L, O)
// rescaled when a round raises M.  The result is either normalised (O / L) to the bf16 output
// rows or stored as one partial again.  The order of summation depends only on t, never on which
// warp does the work, so results are bit-identical from run to run.
struct FoldGeom {
    int ncp, J, g;
    int d0;                         // first element of the lane's first float4 piece
    int dq;                         // elements between its consecutive pieces
};

__device__ __forceinline__ FoldGeom fold_geometry(int ncols, int D, int lane)
{
    FoldGeom fg;
    int ncp = 128 / D;                           // D = 64: at least two rows, so a lane owns a whole float4
    while (ncp < ncols) ncp *= 2;
    fg.ncp = ncp;
    fg.J = ncp * D / 128;
    const int lanes_per_row = 32 / ncp;
    fg.g = lane / lanes_per_row;
    fg.d0 = (lane % lanes_per_row) * 4;
    fg.dq = lanes_per_row * 4;
    return fg;
}

struct FoldJob {
    int n;                          // partials to fold, in this order
    int cap;                        // partials per round (shared-memory sources: n)
    // partial t of a round that starts at t0 sits in shared memory at base + (t - t0) * stride:
    // rows of `pitch` floats, (m, l) at byte offset ml_off (negative for a fetched partial) ...
    uint32_t base;
    int stride, pitch, ml_off;
    // ... except partial alt_t (if >= 0), which sits at alt_base
    int alt_t;
    uint32_t alt_base;
    int alt_pitch, alt_ml_off;
    // fetch != 0: the partials are in global memory -- number i0 + t * istride of a (request, kv
    // head) whose partial 0 is slot slot_first and whose partial i > 0 is slot 2 * (s_first + i) --
    // and are brought to `base` by bulk copies counted on mbarrier `bar` (phases used so far: uses)
    int fetch, s_first, slot_first, i0, istride;
    uint32_t bar;
    int uses;
    // destination: normalised bf16 rows if out_rows != NULL; else global partial slot dst_slot and,
    // if copy_base != 0, the same partial once more in shared memory
    uint16_t *out_rows;
    int dst_slot;
    uint32_t copy_base;
    int copy_pitch, copy_ml_off;

    __device__ __forceinline__ int slot_of(int t) const
    {
        const int i = i0 + t * istride;
        return i == 0 ? slot_first : 2 * (s_first + i);
    }
};

struct FoldCtx {
    float *part;                    // [slots][16 + 8*D]: (m[8], l[8]), then rows [8][D]
    uint32_t *status;
    int ncols, lane;
    int out_off;                    // elements from a pair's first output row to this lane's first float4 piece
    FoldGeom fg;
};

__device__ __forceinline__ float ld_shared_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// Start the bulk copies of one round (partials t0 .. t0 + cnt - 1) of a job with global sources.
template <int D>
__device__ __forceinline__ void fold_fetch(const FoldJob j, const FoldCtx c, int t0)
{
    const int cnt = min(j.cap, j.n - t0);
    const int row_bytes = c.fg.ncp * D * 4;
    const bool alt_here = j.alt_t >= t0 && j.alt_t < t0 + cnt;
    if (c.lane == 0) mbar_arrive_expect_tx(j.bar, (cnt - (alt_here ? 1 : 0)) * (row_bytes + 64));
    __syncwarp();
    if (c.lane < cnt && t0 + c.lane != j.alt_t) {
        const int slot = j.slot_of(t0 + c.lane);
        const uint32_t dst = j.base - 64 + c.lane * j.stride;    // j.base is where the rows go; (m, l) sit in front of them
        bulk_load_1d(dst, c.part + (size_t)slot * (2 * kMaxGroup + kMaxGroup * D), 64 + row_bytes, j.bar);   // (m, l) and the live rows: one copy
    }
}

// Fold a job and store its result.  With global sources the first round's copies are already on
// their way (fold_fetch).  Returns the number of phases the job's mbarrier has completed, or -1 if
// a bounded wait gave up (nothing is stored then).
template <int D>
__device__ __forceinline__ int fold_finish(const FoldJob j, const FoldCtx c)
{
    const int g = c.fg.g, d0 = c.fg.d0, dq = c.fg.dq, J = c.fg.J;
    float M = -INFINITY, L = 0.f;
    float4 acc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    int uses = j.uses;
#pragma unroll 1
    for (int t0 = 0; t0 < j.n; t0 += j.cap) {
        const int cnt = min(j.cap, j.n - t0);
        if (j.fetch) {
            if (t0 > 0) {
                fence_proxy_async();             // the last round's reads precede this round's copies
                __syncwarp();
                fold_fetch<D>(j, c, t0);
            }
            bool ok = mbar_wait_bounded(j.bar, uses & 1, c.status);
            ok = __all_sync(0xffffffffu, ok);
            ++uses;
            if (!ok) return -1;
        }
        float Mr = -INFINITY;
#pragma unroll 2
        for (int i = 0; i < cnt; ++i) {
            const uint32_t ml = (t0 + i == j.alt_t) ? j.alt_base + j.alt_ml_off : j.base + i * j.stride + j.ml_off;
            Mr = fmaxf(Mr, ld_shared_f32(ml + 4 * g));
        }
        // a column that no partial so far has seen a token for keeps -inf (multi-token steps):
        // exponentials are then taken against 0 and come out 0
        const float Mn = fmaxf(M, Mr);
        const float ref = Mn == -INFINITY ? 0.f : Mn;
        if (t0 > 0) {                            // later rounds: bring what has been summed to the new reference
            const float sc = fast_exp2(M - ref);
            L *= sc;
#pragma unroll
            for (int q = 0; q < 8; ++q) { acc[q].x *= sc; acc[q].y *= sc; acc[q].z *= sc; acc[q].w *= sc; }
        }
        M = Mn;
#pragma unroll 2
        for (int i = 0; i < cnt; ++i) {
            const bool alt = t0 + i == j.alt_t;
            const uint32_t pb = alt ? j.alt_base : j.base + i * j.stride;
            const uint32_t ml = pb + (alt ? j.alt_ml_off : j.ml_off);
            const uint32_t rows = pb + (g * (alt ? j.alt_pitch : j.pitch) + d0) * 4;
            const float f = fast_exp2(ld_shared_f32(ml + 4 * g) - ref);
            L += f * ld_shared_f32(ml + 4 * (kMaxGroup + g));
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (q < J) {
                    const float4 a = ld_shared_f32x4(rows + q * dq * 4);
                    acc[q].x += f * a.x; acc[q].y += f * a.y; acc[q].z += f * a.z; acc[q].w += f * a.w;
                }
            }
        }
        __syncwarp();                            // every lane has read the round before anything overwrites it
    }
    if (j.out_rows != nullptr) {
        if (g < c.ncols) {
            const float inv = __frcp_rn(L);
            uint16_t *row = j.out_rows + c.out_off;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (q < J) {
                    uint2 packed;
                    packed.x = pack_bf16x2(acc[q].x * inv, acc[q].y * inv);
                    packed.y = pack_bf16x2(acc[q].z * inv, acc[q].w * inv);
                    *(uint2 *)(row + q * dq) = packed;
                }
            }
        }
    } else {
        float *slot = c.part + (size_t)j.dst_slot * (2 * kMaxGroup + kMaxGroup * D);
        float *rows = slot + 2 * kMaxGroup + g * D + d0;
#pragma unroll
        for (int q = 0; q < 8; ++q)
            if (q < J) *(float4 *)(rows + q * dq) = acc[q];
        if (d0 == 0) {
            slot[g] = M;
            slot[kMaxGroup + g] = L;
        }
        if (j.copy_base != 0) {
            const uint32_t crow = j.copy_base + (g * j.copy_pitch + d0) * 4;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q < J)
                    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(crow + q * dq * 4), "f"(acc[q].x), "f"(acc[q].y),
                                 "f"(acc[q].z), "f"(acc[q].w) : "memory");
            if (d0 == 0) {
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(j.copy_base + j.copy_ml_off + 4 * g), "f"(M) : "memory");
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(j.copy_base + j.copy_ml_off + 4 * (kMaxGroup + g)), "f"(L) : "memory");
            }
            __syncwarp();
        }
    }
    return uses;
}

template <int D, int W, int NS>
struct AttnLayout {
    static constexpr int kHalves = D / 64;                       // 128-byte column blocks per row
    static constexpr int kHalfBytes = 32 * 128;                  // one TMA box: 32 rows x 128 B
    static constexpr int kPageBytes = kHalves * kHalfBytes;      // K and V rows of one (page, head)
    static constexpr int kStageBytes = kPagesPerTile * kPageBytes;
    static constexpr int kKSteps = D / 16;
    static constexpr int kDTiles = D / 16;
    static constexpr int kStagePitch = D + 4;                    // floats per staging row (bank spread)
    static constexpr int kStagingBytes = (kMaxGroup * kStagePitch + 2 * kMaxGroup) * 4;   // rows, then m[8], l[8]
    static constexpr int kParkBytes = (kMaxGroup * D + 2 * kMaxGroup) * 4;                // the same, rows unpadded
    static constexpr int kRingBytes = W * NS * kStageBytes;
    static constexpr int kStagingOff = kRingBytes;
    static constexpr int kParkOff = kStagingOff + W * kStagingBytes;
    static constexpr int kBarOff = kParkOff + W * kParkBytes;
    static constexpr int kCtrOff = kBarOff + W * NS * 8;                                  // W counters of the CTA stage
    static constexpr int kSmemBytes = kCtrOff + W * 4 + 1024;
    static constexpr int kThreads = W * 32;
};

// A cursor over the tiles of a span.  The issue cursor and the compute cursor are two copies.
struct SpanCursor {
    int r, h, tile;       // next tile: request, kv head, tile within (r, h)
    int L, tiles;         // length and tile count of request r
    long long v;          // unit index of that tile on the plan's axis

    // step to the next tile; returns false when it left the last request
    __device__ __forceinline__ bool next(const AttnParams &p)
    {
        ++v;
        if (++tile < tiles) return true;
        tile = 0;
        v += kPieceCostTiles;                 // the next (request, kv head) starts with its overhead units
        if (++h < p.num_kv_heads) return true;
        h = 0;
        do {
            if (++r >= p.batch) return false;
            L = __ldg(p.seq_lens + r);
            tiles = tiles_of_length(L, p.max_pages_per_req, p.q_len);
        } while (tiles == 0);
        return true;
    }
};

// kMulti = false: one new token per request (every live column sees the whole context);
// kMulti = true:  q_len > 1 new tokens, each column with its own causal limit.
template <int D, int W, int NS, bool kMulti>
__global__ void __launch_bounds__(W * 32, 1)
paged_decode_attn_kernel(const __grid_constant__ CUtensorMap tmap, const AttnParams p)
{
    using Lay = AttnLayout<D, W, NS>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int span = blockIdx.x * W + warp;

    const uint32_t ring = smem_u32(smem) + warp * NS * Lay::kStageBytes;
    float *staging = (float *)(smem + Lay::kStagingOff + warp * Lay::kStagingBytes);
    float *park = (float *)(smem + Lay::kParkOff + warp * Lay::kParkBytes);
    const uint32_t bars = smem_u32(smem + Lay::kBarOff) + warp * NS * 8;
    int *cta_ctr = (int *)(smem + Lay::kCtrOff);

    if (threadIdx.x < W) cta_ctr[threadIdx.x] = 0;
    __syncthreads();                             // the only CTA-wide barrier: the counters of the CTA stage are zero
    if (span >= p.num_spans) return;
    unsigned long long t_start = 0;
    if (lane == 0) {
        t_start = global_timer_ns();
        prefetch_tensormap(&tmap);
        for (int s = 0; s < NS; ++s) mbar_init(bars + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncwarp();
    if (p.early_loads < 0) grid_dependency_wait();

    // ---- plan: where does this warp's span start?
    // Nothing read up to the dependency wait below is written by the preceding kernel of a decode
    // step (the KV append writes only the pool), so this prologue overlaps that kernel's tail.
    const SpanStart st = warp_plan(p.seq_lens, p.batch, p.max_pages_per_req, p.num_kv_heads, p.num_spans, span, lane,
                                   p.q_len);
    if (st.r < 0 || span == 0) {
        grid_dependency_wait();
        grid_launch_dependents();
        if (span == 0)
            flag_unusable_requests(p.seq_lens, p.batch, p.max_pages_per_req, p.q_len, lane, p.out,
                                   p.q_len * p.num_q_heads * D, p.status);
    }
    if (st.r < 0) {
        if (lane == 0) {
            p.span_start[span] = make_int4(-1, -1, -1, -1);
            p.trace[span * 8 + 0] = t_start;
            p.trace[span * 8 + 1] = 0;
        }
        if (lane == 0) p.trace[span * 8 + 2] = p.trace[span * 8 + 3] = global_timer_ns();
        return;
    }
    const long long v_end = st.end;
    const int q_span = st.q;
    const int G = p.group;
    const int ncols = G * p.q_pass;              // live MMA columns: column c = new token q_base + c / G, head c % G
    const int qi_stride = p.num_q_heads * D;     // elements between a request's consecutive new tokens in q / out

    // ---- issue side: block-table entries travel in registers, 32 pages (16 tiles) per chunk
    SpanCursor ic;
    ic.r = st.r; ic.h = st.h; ic.tile = st.tile; ic.L = st.L; ic.tiles = st.tiles_r; ic.v = st.v;
    bool more_to_issue = true;                   // the issue cursor still points at a tile of this span
    int issued = 0, i_slot = 0;                  // i_slot = issued % NS
    bool alive = true;
    auto table_row = [&](int r) { return p.block_tables + (size_t)r * p.max_pages_per_req; };
    auto load_chunk = [&](int r, int chunk) -> int {
        const int idx = chunk * 32 + lane;
        return (r < p.batch && idx < p.max_pages_per_req) ? __ldg(table_row(r) + idx) : -1;
    };
    constexpr int kTilesPerChunk = 32 / kPagesPerTile;
    int cur_chunk = ic.tile / kTilesPerChunk;
    int cur_val = load_chunk(ic.r, cur_chunk);
    int nxt_val = load_chunk(ic.r, cur_chunk + 1);
    // chunk 0 of the row the NEXT (request, kv head) will read: this row again, or the next request's
    int pf_row = (ic.h + 1 < p.num_kv_heads) ? ic.r : ic.r + 1;
    int pf_val = load_chunk(pf_row, 0);

    // query fragments of a (request, kv head), fetched when the issue cursor enters it
    uint32_t qn[Lay::kKSteps][2];
    int qn_r = -1, qn_h = -1;
    const int c_row = lane >> 2;                 // the column this lane loads Q for
    auto load_q = [&](uint32_t (&dst)[Lay::kKSteps][2], int r, int h) {
        const uint32_t *qrow = (const uint32_t *)(p.q + ((size_t)r * p.q_len + p.q_base + c_row / G) * qi_stride +
                                                  (size_t)(h * G + c_row % G) * D);
#pragma unroll
        for (int ks = 0; ks < Lay::kKSteps; ++ks) {
            dst[ks][0] = c_row < ncols ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
            dst[ks][1] = c_row < ncols ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
        }
    };

    // Issue the loads of the tile under the issue cursor into stage issued % NS, then advance.
    // rows of the (request, kv head) whose last tile is in flight: lane l < 2*d/8 holds 16 bytes of
    // the key row (first d/8 lanes) or of the value row
    constexpr int kRowVecs = D / 8;
    uint4 an_val = make_uint4(0u, 0u, 0u, 0u);
    int an_r = -1, an_h = -1, an_page = -1;
    auto load_new_rows = [&](int r, int h) -> uint4 {
        if (lane >= 2 * kRowVecs) return make_uint4(0u, 0u, 0u, 0u);
        const uint4 *src = (lane < kRowVecs ? p.k_new : p.v_new) + ((size_t)r * p.num_kv_heads + h) * kRowVecs;
        return __ldg(src + (lane % kRowVecs));
    };
#ifdef CKV_TRACE_WAITS
    unsigned long long t_issue = 0, t_masked = 0;
#endif
    bool inputs_ready = true;                    // q, k_new and v_new may be read (the dependency wait is behind us)
    const uint64_t kv_policy = l2_evict_first_policy();
    auto issue_next = [&]() {
#ifdef CKV_TRACE_WAITS
        const unsigned long long i0 = global_timer_ns();
#endif
        const int ck = ic.tile / kTilesPerChunk;
        if (ck != cur_chunk) {
            cur_chunk = ck;
            cur_val = nxt_val;
            nxt_val = load_chunk(ic.r, ck + 1);
        }
        const int n_pages = (ic.L + kPageSize - 1) / kPageSize;
        const int np = min(kPagesPerTile, n_pages - ic.tile * kPagesPerTile);
        const int pg = lane / Lay::kHalves, hf = lane % Lay::kHalves;
        int page = __shfl_sync(0xffffffffu, cur_val, ((ic.tile % kTilesPerChunk) * kPagesPerTile + pg) & 31);
        const int slot = i_slot;
        if (++i_slot == NS) i_slot = 0;
        // The stage's previous contents were read by this warp's ldmatrix instructions, whose results
        // have all been consumed by MMAs earlier in program order, so the reads are complete.
        if (lane == 0) mbar_arrive_expect_tx(bars + slot * 8, np * Lay::kPageBytes);
        __syncwarp();
        if (lane < np * Lay::kHalves) {
            int src_page = page;
            if (page < 0 || page >= p.num_pages) {
                atomicOr(p.status, kStatusBadPage);
                src_page = 0;
            }
            const int y = ((p.layer_page_base + src_page) * p.num_kv_heads + ic.h) * 32;
            tma_load_2d(ring + slot * Lay::kStageBytes + pg * Lay::kPageBytes + hf * Lay::kHalfBytes,
                        &tmap, hf * 64, y, bars + slot * 8, kv_policy);
        }
        if (p.k_new != nullptr && ic.tile == ic.tiles - 1 && an_r < 0 && inputs_ready) {
            // last tile of this (request, kv head): fetch the rows to append and remember their page
            const bool bad = page < 0 || page >= p.num_pages;               // before any redirect above
            an_val = load_new_rows(ic.r, ic.h);
            an_page = __shfl_sync(0xffffffffu, bad ? -1 : page, (np - 1) * Lay::kHalves);
            an_r = ic.r; an_h = ic.h;
        }
        ++issued;
        more_to_issue = ic.next(p) && ic.v < v_end;
        if (more_to_issue) {
            if (ic.tile == 0) {
                // entered a new (request, kv head): its first table chunk was fetched ahead
                cur_chunk = 0;
                cur_val = (pf_row == ic.r) ? pf_val : load_chunk(ic.r, 0);
                nxt_val = load_chunk(ic.r, 1);
                pf_row = (ic.h + 1 < p.num_kv_heads) ? ic.r : ic.r + 1;
                pf_val = (pf_row == ic.r) ? cur_val : load_chunk(pf_row, 0);
                if (qn_r < 0 && inputs_ready) {
                    load_q(qn, ic.r, ic.h);
                    qn_r = ic.r; qn_h = ic.h;
                }
            }
        }
#ifdef CKV_TRACE_WAITS
        t_issue += global_timer_ns() - i0;
#endif
    };

    // A step with the fused append is the only writer of its layer's pool, so its first loads can
    // start before the preceding kernel has finished -- under that kernel's tail -- as long as
    // nothing of q, k_new or v_new is touched yet and no tile is fetched that the preceding kernel
    // may still be writing.  If that kernel is the previous decode step of this layer, it writes
    // each request's previous last position, L-2 as seen from this step (this step's own row, L-1,
    // is put into the staged tile before use, so its copy may race with the store).  Tiles that
    // hold a position >= L-2 therefore stay behind the dependency wait.  The dependents of this
    // kernel are released only after the wait, so a kernel's early loads overlap its immediate
    // predecessor and nothing older.
    const bool early = p.k_new != nullptr && p.early_loads > 0;
    if (early) {
        inputs_ready = false;
        while (issued < NS && more_to_issue && ic.tile < (ic.L - 2) / kTileTokens) issue_next();
        inputs_ready = true;
    }
    grid_dependency_wait();                       // the workspace, q, the new rows and `out` are ours from here on
    grid_launch_dependents();
    if (lane == 0) {
        p.span_start[span] = make_int4(st.r, st.h, st.tile, (int)st.v);
        p.trace[span * 8 + 0] = t_start;
        p.trace[span * 8 + 1] = 0;
    }
    while (issued < NS && more_to_issue) issue_next();

    // ---- compute side
    SpanCursor cc;
    cc.r = st.r; cc.h = st.h; cc.tile = st.tile; cc.L = st.L; cc.tiles = st.tiles_r; cc.v = st.v;
    const int g0 = (lane & 3) * 2;               // first of the two group columns this lane accumulates
    const int qi0 = g0 / G, qi1 = (g0 + 1) / G;  // the new tokens those two columns belong to
    uint32_t k_off[4], v_off[4];                 // ldmatrix lane offsets inside one page block
    {
        const int krow = (lane & 7) + ((lane >> 3) & 1) * 8;          // key row for matrices 0..3
        const int ksel = lane >> 4;                                    // second 16-byte chunk of the k16 step
        const int vrow = 16 + (lane & 7) + (lane >> 4) * 8;           // value rows follow the 16 key rows
        const int vsel = (lane >> 3) & 1;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            k_off[j] = krow * 128 + (((j * 2 + ksel) ^ (lane & 7)) << 4);
            v_off[j] = vrow * 128 + (((j * 2 + vsel) ^ (lane & 7)) << 4);
        }
    }

    int done = 0;                                // tiles computed (or skipped after a wait gave up)
    int c_slot = 0;                              // done % NS and the parity of done / NS, kept without divisions
    uint32_t c_phase = 0;
    int landed = 0;                              // tiles whose copies were seen to complete
    bool more_to_compute = true;
    unsigned long long t_wait = 0, t_between = 0, t_piece_end = 0;
    int n_pieces = 0;
    bool first_piece = true;
    // a span writes at most two partials: its first piece and its last piece
    int pend_first[2] = {-1, -1}, pend_last[2] = {0, 0};
    uint16_t *pend_out[2] = {nullptr, nullptr};
    while (more_to_compute) {
        const int n = (int)min((long long)(cc.tiles - cc.tile), v_end - cc.v);
        const bool complete = (cc.tile == 0 && n == cc.tiles);
        const int piece_r = cc.r, piece_h = cc.h, piece_L = cc.L, piece_tile0 = cc.tile, piece_tiles = cc.tiles;

        ++n_pieces;
        uint32_t qf[Lay::kKSteps][2];
        if (qn_r == piece_r && qn_h == piece_h) {
#pragma unroll
            for (int ks = 0; ks < Lay::kKSteps; ++ks) { qf[ks][0] = qn[ks][0]; qf[ks][1] = qn[ks][1]; }
            qn_r = -1;
        } else {
            load_q(qf, piece_r, piece_h);
        }
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[Lay::kDTiles][4];
#pragma unroll
        for (int dt = 0; dt < Lay::kDTiles; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;

        for (int ti = piece_tile0; ti < piece_tile0 + n; ++ti, ++done) {
            const int slot = c_slot;
            const uint32_t phase = c_phase;
            if (++c_slot == NS) { c_slot = 0; c_phase ^= 1u; }
            if (alive) {
#ifdef CKV_TRACE_WAITS
                const unsigned long long w0 = global_timer_ns();
#endif
                alive = mbar_wait_bounded(bars + slot * 8, phase, p.status);
                alive = __all_sync(0xffffffffu, alive);
#ifdef CKV_TRACE_WAITS
                t_wait += global_timer_ns() - w0;
#endif
            }
            if (!alive) continue;
#ifdef CKV_TRACE_WAITS
            const unsigned long long w1 = global_timer_ns();
#endif
            ++landed;
            if (done == 0 && lane == 0) p.trace[span * 8 + 1] = global_timer_ns();

            const int ntok = min(kTileTokens, piece_L - ti * kTileTokens);      // tokens of the context in this tile
            // Causality among the step's new tokens: column c (new token t = q_base + c / G) sees the
            // context up to and including its own position, i.e. vis_all + t tokens; every column sees vis_all.
            const int vis_all = kMulti ? piece_L - p.q_len + 1 : piece_L;
            const bool full_tile = (ti + 1) * kTileTokens <= vis_all;
            const int lim0 = kMulti ? min(ntok, vis_all + p.q_base + qi0 - ti * kTileTokens) : ntok;   // visible tokens of this tile,
            const int lim1 = kMulti ? min(ntok, vis_all + p.q_base + qi1 - ti * kTileTokens) : ntok;   // for this lane's two columns
            const int np = (ntok + kPageSize - 1) / kPageSize;
            const uint32_t sb = ring + slot * Lay::kStageBytes;

            if (!full_tile && (ntok & (kPageSize - 1))) {
                // Value rows past the context's end hold whatever the pool holds; their weights are
                // zero, but 0 * NaN would poison the sum, so clear them in shared memory.
                const int lp = np - 1, row0 = ntok - lp * kPageSize;
                const int pieces = (kPageSize - row0) * 8 * Lay::kHalves;
                for (int i = lane; i < pieces; i += 32) {
                    const int hf = i / ((kPageSize - row0) * 8);
                    const int rem = i % ((kPageSize - row0) * 8);
                    const uint32_t a = sb + lp * Lay::kPageBytes + hf * Lay::kHalfBytes +
                                       (16 + row0 + rem / 8) * 128 + (rem % 8) * 16;
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                }
                fence_proxy_async();              // these generic-proxy writes precede the stage's next TMA fill
                __syncwarp();
            }

            if (p.k_new != nullptr && ti == piece_tiles - 1) {
                // this warp owns the append of (piece_r, piece_h): position L-1 is in the tile's last page
                uint4 val;
                int page;
                if (an_r == piece_r && an_h == piece_h) {
                    val = an_val; page = an_page; an_r = -1;
                } else {                                                     // not fetched ahead (very short contexts)
                    val = load_new_rows(piece_r, piece_h);
                    page = __ldg(table_row(piece_r) + (piece_L - 1) / kPageSize);
                    if (page < 0 || page >= p.num_pages) page = -1;
                }
                const int pos_slot = (piece_L - 1) % kPageSize;
                if (lane < 2 * kRowVecs) {
                    const int kv = lane / kRowVecs, vec = lane % kRowVecs;
                    if (page >= 0) {
                        const size_t row = (((size_t)page * p.num_kv_heads + piece_h) * 2 + kv) * kPageSize + pos_slot;
                        p.pool_layer[row * kRowVecs + vec] = val;
                    } else {
                        atomicOr(p.status, kStatusBadPage);
                    }
                    const uint32_t a = sb + (np - 1) * Lay::kPageBytes + (vec / 8) * Lay::kHalfBytes +
                                       (kv * 16 + pos_slot) * 128 + (((vec % 8) ^ (pos_slot & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
                }
                fence_proxy_async();              // generic-proxy writes precede the stage's next TMA fill
                __syncwarp();
            }

            // ---- S^T = K Q^T
            float s[kPagesPerTile][4];
#pragma unroll
            for (int mt = 0; mt < kPagesPerTile; ++mt) s[mt][0] = s[mt][1] = s[mt][2] = s[mt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < Lay::kKSteps; ++ks) {
#pragma unroll
                for (int mt = 0; mt < kPagesPerTile; ++mt) {
                    if (full_tile || mt < np) {
                        uint32_t a[4];
                        ldmatrix_x4(a, sb + mt * Lay::kPageBytes + (ks / 4) * Lay::kHalfBytes + k_off[ks % 4]);
                        mma_bf16_16816(s[mt], a, qf[ks][0], qf[ks][1]);
                    }
                }
            }

            // ---- online softmax in the log2 domain.  Scores stay unscaled: the scale rides in the
            // FMA that forms the exponent, and a maximum is scaled once (the scale is positive).
            if (!full_tile) {
#pragma unroll
                for (int mt = 0; mt < kPagesPerTile; ++mt) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tok = mt * kPageSize + (lane >> 2) + (i >= 2 ? 8 : 0);
                        if (!(tok < ((i & 1) ? lim1 : lim0))) s[mt][i] = -INFINITY;      // selected, never multiplied
                    }
                }
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int mt = 0; mt < kPagesPerTile; ++mt) {
                mx0 = fmaxf(mx0, fmaxf(s[mt][0], s[mt][2]));
                mx1 = fmaxf(mx1, fmaxf(s[mt][1], s[mt][3]));
            }
            mx0 *= p.scale_log2;
            mx1 *= p.scale_log2;
            // The reference a column's exponentials are taken against only has to be near its maximum:
            // it moves (with the reduction across lanes and the rescale that this costs) only when
            // some score of the tile exceeds it by more than 2^8.
            float mn0 = m0, mn1 = m1;
            if (__any_sync(0xffffffffu, mx0 > m0 + 8.f || mx1 > m1 + 8.f)) {
#pragma unroll
                for (int x = 4; x < 32; x <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, x));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, x));
                }
                const float mo0 = m0, mo1 = m1;
                mn0 = fmaxf(mo0, mx0); mn1 = fmaxf(mo1, mx1);
                m0 = mn0; m1 = mn1;
                if (kMulti) {
                    mn0 = (mn0 == -INFINITY) ? 0.f : mn0;
                    mn1 = (mn1 == -INFINITY) ? 0.f : mn1;
                }
                const float al0 = fast_exp2(mo0 - mn0), al1 = fast_exp2(mo1 - mn1);
                l0 *= al0; l1 *= al1;
#pragma unroll
                for (int dt = 0; dt < Lay::kDTiles; ++dt) {
                    o[dt][0] *= al0; o[dt][2] *= al0;
                    o[dt][1] *= al1; o[dt][3] *= al1;
                }
            } else if (kMulti) {
                mn0 = (mn0 == -INFINITY) ? 0.f : mn0;
                mn1 = (mn1 == -INFINITY) ? 0.f : mn1;
            }
            uint32_t pb[kPagesPerTile][2];
#pragma unroll
            for (int mt = 0; mt < kPagesPerTile; ++mt) {
                const float p0 = fast_exp2(fmaf(s[mt][0], p.scale_log2, -mn0)), p1 = fast_exp2(fmaf(s[mt][1], p.scale_log2, -mn1));
                const float p2 = fast_exp2(fmaf(s[mt][2], p.scale_log2, -mn0)), p3 = fast_exp2(fmaf(s[mt][3], p.scale_log2, -mn1));
                l0 += p0 + p2;
                l1 += p1 + p3;
                pb[mt][0] = movmatrix_trans(pack_bf16x2(p0, p1));       // tokens 0..7 of the page
                pb[mt][1] = movmatrix_trans(pack_bf16x2(p2, p3));       // tokens 8..15
            }

            // ---- O^T += V^T P^T
#pragma unroll
            for (int dt = 0; dt < Lay::kDTiles; ++dt) {
#pragma unroll
                for (int mt = 0; mt < kPagesPerTile; ++mt) {
                    if (full_tile || mt < np) {
                        uint32_t a[4];
                        ldmatrix_x4_trans(a, sb + mt * Lay::kPageBytes + (dt / 4) * Lay::kHalfBytes + v_off[dt % 4]);
                        mma_bf16_16816(o[dt], a, pb[mt][0], pb[mt][1]);
                    }
                }
            }
#ifdef CKV_TRACE_WAITS
            if (ti == piece_tile0 && !first_piece) t_masked += global_timer_ns() - w1;
#endif
            // the stage is free again: refill it with the tile NS ahead
            if (more_to_issue) issue_next();
        }
        t_piece_end = global_timer_ns();

        // ---- finish the piece: row sums across the warp, then through the staging tile
#pragma unroll
        for (int x = 4; x < 32; x <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, x);
            l1 += __shfl_xor_sync(0xffffffffu, l1, x);
        }
#pragma unroll
        for (int dt = 0; dt < Lay::kDTiles; ++dt) {
            const int d = dt * 16 + (lane >> 2);
            staging[g0 * Lay::kStagePitch + d] = o[dt][0];
            staging[(g0 + 1) * Lay::kStagePitch + d] = o[dt][1];
            staging[g0 * Lay::kStagePitch + d + 8] = o[dt][2];
            staging[(g0 + 1) * Lay::kStagePitch + d + 8] = o[dt][3];
        }
        __syncwarp();
        uint16_t *out_rows = p.out + ((size_t)piece_r * p.q_len + p.q_base) * qi_stride + (size_t)piece_h * G * D;
        if (complete) {
#pragma unroll
            for (int g = 0; g < kMaxGroup; ++g) {
                const float lg = __shfl_sync(0xffffffffu, (g & 1) ? l1 : l0, g >> 1);
                if (g < ncols && lane * 4 < D) {
                    const float4 a = *(const float4 *)(staging + g * Lay::kStagePitch + lane * 4);
                    const float inv = 1.f / lg;
                    uint2 packed;
                    packed.x = pack_bf16x2(a.x * inv, a.y * inv);
                    packed.y = pack_bf16x2(a.z * inv, a.w * inv);
                    *(uint2 *)(out_rows + (size_t)(g / G) * qi_stride + (size_t)(g % G) * D + lane * 4) = packed;
                }
            }
        } else {
            // The partial stays in shared memory until the span has been streamed.  A piece whose
            // (request, kv head) began in an earlier span is this span's first piece: it moves to the
            // parking buffer, since the staging tile is reused.  A piece whose pair begins here and
            // runs on into the next span is the span's last piece and stays in the staging tile.
            const bool entered = piece_tile0 > 0;
            float *dst_ml = entered ? park + kMaxGroup * D : staging + kMaxGroup * Lay::kStagePitch;
            if (entered) {
#pragma unroll
                for (int g = 0; g < kMaxGroup; ++g)
                    if (lane * 4 < D)
                        *(float4 *)(park + g * D + lane * 4) = *(const float4 *)(staging + g * Lay::kStagePitch + lane * 4);
            }
            if (lane < 4) {
                dst_ml[g0] = m0; dst_ml[g0 + 1] = m1;
                dst_ml[kMaxGroup + g0] = l0; dst_ml[kMaxGroup + g0 + 1] = l1;
            }
            // ---- remember the piece; it is handed on once the whole span has been streamed, so that
            // neither a fence nor a merge ever interrupts this warp's loads
            const long long tile0_unit = cc.v - piece_tile0;             // unit of this (request, kv head)'s tile 0
            const int k = entered ? 0 : 1;
            pend_first[k] = (int)(tile0_unit / q_span);                   // first and last span that hold its tiles
            pend_last[k] = (int)((tile0_unit + piece_tiles - 1) / q_span);
            pend_out[k] = out_rows;
        }
        __syncwarp();                             // staging is reused by the next piece
        t_between += global_timer_ns() - t_piece_end;
        first_piece = false;
        // move the compute cursor past the piece: to the next (request, kv head) or out of the span
        cc.tile += n - 1;
        cc.v += n - 1;
        more_to_compute = cc.next(p) && cc.v < v_end;
    }

    if (lane == 0) p.trace[span * 8 + 2] = global_timer_ns();

    // ---- hand-over.  Every merge below is one FoldJob run by fold_finish.
    //
    // CTA stage: consecutive spans belong to the warps of one CTA, so the partials of a (request,
    // kv head) that several of this CTA's warps hold are folded straight from shared memory: each
    // warp counts itself in on a shared counter once its span has been streamed, and the last one
    // does the fold (wait-free, no global round trip).  If the pair lies inside this CTA the result
    // is final; otherwise it is the CTA's one partial of the pair: it goes to global memory and,
    // once more, into this warp's own buffer.
    // Grid stage, in units of CTAs: the CTA that arrives last for a pair (a counter in global
    // memory) fetches the other CTAs' partials into its idle ring with bulk copies and folds them
    // with its own; a pair cut into more than kTreeFrom partials is folded in two levels.
    FoldCtx fc;
    fc.part = p.part; fc.status = p.status;
    fc.ncols = ncols; fc.lane = lane;
    fc.fg = fold_geometry(ncols, D, lane);
    fc.out_off = (fc.fg.g / G) * qi_stride + (fc.fg.g % G) * D + fc.fg.d0;
    const uint32_t staging_u32 = smem_u32(smem + Lay::kStagingOff), park_u32 = smem_u32(smem + Lay::kParkOff);
    constexpr int kStagingMl = kMaxGroup * Lay::kStagePitch * 4, kParkMl = kMaxGroup * D * 4;
    const int part_bytes = fc.fg.ncp * D * 4 + 64;               // a fetched partial in the ring: (m, l), then the live rows
    int bar_uses[2] = {(done + NS - 1) / NS, (done + NS - 2) / NS};   // phases the first two stage barriers have completed
    FoldJob jobs[2];
    int n_jobs = 0;
    int tree_first[2] = {-1, -1}, tree_last[2] = {0, 0};         // pairs that take the counter protocol for more than two CTAs
    uint16_t *tree_out[2] = {nullptr, nullptr};
    uint32_t tree_buf[2] = {0u, 0u};
    auto grid_job = [&](int c_first, int n, int i0, int istride, int alt_t, uint32_t buf, bool in_staging) {
        FoldJob j;
        j.n = n; j.cap = 1;                       // the ring region and cap are set when the jobs are started
        j.base = 0; j.stride = part_bytes; j.pitch = D; j.ml_off = -64;   // as fetched: (m, l), then the rows at `base`
        j.alt_t = alt_t; j.alt_base = buf;
        j.alt_pitch = in_staging ? Lay::kStagePitch : D; j.alt_ml_off = in_staging ? kStagingMl : kParkMl;
        j.fetch = 1; j.s_first = c_first; j.slot_first = 2 * c_first + 1; j.i0 = i0; j.istride = istride;
        j.bar = 0; j.uses = 0;
        j.out_rows = nullptr; j.dst_slot = 0; j.copy_base = 0; j.copy_pitch = 0; j.copy_ml_off = 0;
        return j;
    };
    {
        const int b0 = blockIdx.x * W;
#pragma unroll 1                                      // executed once per warp: keep the code small
        for (int k = 0; k < 2 && alive; ++k) {
            if (pend_first[k] < 0) continue;
            const int f = pend_first[k], l = pend_last[k];
            const int fb = max(f, b0), lb = min(l, b0 + W - 1), cb = lb - fb + 1;
            if (cb > 1) {
                __threadfence_block();
                __syncwarp();
                int prior = 0;
                if (lane == 0) prior = atomicAdd(cta_ctr + (fb - b0), 1);
                prior = __shfl_sync(0xffffffffu, prior, 0);
                if (prior != cb - 1) continue;    // a later warp of this CTA folds them
                __threadfence_block();
            }
            // the partials of spans fb..lb: span f keeps its own in its staging tile, the others
            // (which the pair entered from the left) in their parking buffers
            const uint32_t my_buf = k == 0 ? park_u32 + warp * Lay::kParkBytes : staging_u32 + warp * Lay::kStagingBytes;
            FoldJob j;
            j.n = cb; j.cap = cb;
            j.base = park_u32 + (fb - b0) * Lay::kParkBytes; j.stride = Lay::kParkBytes; j.pitch = D; j.ml_off = kParkMl;
            j.alt_t = f >= fb ? 0 : -1;
            j.alt_base = staging_u32 + (fb - b0) * Lay::kStagingBytes; j.alt_pitch = Lay::kStagePitch; j.alt_ml_off = kStagingMl;
            j.fetch = 0; j.s_first = 0; j.slot_first = 0; j.i0 = 0; j.istride = 1; j.bar = 0; j.uses = 0;
            j.out_rows = nullptr; j.dst_slot = 0; j.copy_base = 0; j.copy_pitch = 0; j.copy_ml_off = 0;
            const int c_first = f / W, c_last = l / W;
            if (c_first == c_last) {              // the pair lies inside this CTA: done
                j.out_rows = pend_out[k];
                fold_finish<D>(j, fc);
                continue;
            }
            // partial 0 of a pair (the CTA it begins in) lives in that CTA's odd slot, the others in
            // the even slot of their CTA
            j.dst_slot = (int)blockIdx.x == c_first ? 2 * (int)blockIdx.x + 1 : 2 * (int)blockIdx.x;
            if (cb > 1) {                         // keep the folded partial here as well
                j.copy_base = my_buf;
                j.copy_pitch = k == 0 ? D : Lay::kStagePitch;
                j.copy_ml_off = k == 0 ? kParkMl : kStagingMl;
            }
            fold_finish<D>(j, fc);                // publish: the stores drain while the counters are asked
            tree_first[k] = c_first; tree_last[k] = c_last; tree_out[k] = pend_out[k]; tree_buf[k] = my_buf;
        }
    }

    // ---- arrival of this CTA's partials (both pairs together: two round trips in all).
    // A pair shared by two CTAs first asks its counter with a compare-and-swap: if the other CTA has
    // arrived already (counter at 1) this warp is the last and takes the counter back to 0 in the
    // same operation.  The fence that publishes this warp's partials runs while those are in flight.
    // Everybody else then counts itself in; whoever brings a counter to its full count is the last.
    if (alive && (tree_first[0] >= 0 || tree_first[1] >= 0)) {
        int n_part[2], sub[2], grp[2], grp_cnt[2], n_grp[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            n_part[k] = tree_first[k] >= 0 ? tree_last[k] - tree_first[k] + 1 : 0;
            sub[k] = 0; grp[k] = 0; grp_cnt[k] = n_part[k]; n_grp[k] = 1;
            if (n_part[k] > kTreeFrom) {
                sub[k] = merge_group_size(n_part[k]);
                grp[k] = ((int)blockIdx.x - tree_first[k]) / sub[k];
                n_grp[k] = (n_part[k] + sub[k] - 1) / sub[k];
                grp_cnt[k] = min(sub[k], n_part[k] - grp[k] * sub[k]);
            }
        }
        int seen0 = 0, seen1 = 0;
        if (lane == 0) {
            if (n_part[0] == 2) seen0 = atomicCAS(p.arrivals + tree_first[0], 1, 0);
            if (n_part[1] == 2) seen1 = atomicCAS(p.arrivals + tree_first[1], 1, 0);
        }
        __threadfence();                          // the partials' stores have left; what the other CTAs published is visible
        __syncwarp();
        seen0 = __shfl_sync(0xffffffffu, seen0, 0);
        seen1 = __shfl_sync(0xffffffffu, seen1, 0);
        bool last[2];
        last[0] = n_part[0] == 2 && seen0 == 1;
        last[1] = n_part[1] == 2 && seen1 == 1;
        int prior0 = -1, prior1 = -1;
        if (lane == 0) {                          // both round trips in flight together
            if (tree_first[0] >= 0 && !last[0]) prior0 = atomicAdd(p.arrivals + tree_first[0] + (sub[0] ? 1 + grp[0] : 0), 1);
            if (tree_first[1] >= 0 && !last[1]) prior1 = atomicAdd(p.arrivals + tree_first[1] + (sub[1] ? 1 + grp[1] : 0), 1);
        }
        prior0 = __shfl_sync(0xffffffffu, prior0, 0);
        prior1 = __shfl_sync(0xffffffffu, prior1, 0);
        const bool late0 = prior0 >= 0 && prior0 == grp_cnt[0] - 1, late1 = prior1 >= 0 && prior1 == grp_cnt[1] - 1;
        if (late0 || late1) {
            __threadfence();
            if (lane == 0) {                      // counters are ready for the next launch
                if (late0) p.arrivals[tree_first[0] + (sub[0] ? 1 + grp[0] : 0)] = 0;
                if (late1) p.arrivals[tree_first[1] + (sub[1] ? 1 + grp[1] : 0)] = 0;
            }
        }
        last[0] = last[0] || late0;
        last[1] = last[1] || late1;
#pragma unroll 1
        for (int k = 0; k < 2 && alive; ++k) {
            if (!last[k]) continue;
            const int me = (int)blockIdx.x - tree_first[k];
            if (sub[k] == 0) {                    // one level: this CTA's partial is still in its own buffer
                jobs[n_jobs] = grid_job(tree_first[k], n_part[k], 0, 1, me, tree_buf[k], k == 1);
                jobs[n_jobs].out_rows = tree_out[k];
                ++n_jobs;
                continue;
            }
            // first level of a two-level merge: fold this group's partials into the slot of its first
            // member, right away and with the whole ring; then count the group in
            FoldJob j = grid_job(tree_first[k], grp_cnt[k], grp[k] * sub[k], 1, me - grp[k] * sub[k], tree_buf[k], k == 1);
            j.dst_slot = j.slot_of(0);
            j.base = ring + 64; j.cap = min(32, NS * Lay::kStageBytes / part_bytes);
            j.bar = bars; j.uses = bar_uses[0];
            fence_proxy_async();                  // partials written through the generic proxy, read by bulk copies
            fold_fetch<D>(j, fc, 0);
            const int u = fold_finish<D>(j, fc);
            if (u < 0) { alive = false; break; }
            bar_uses[0] = u;
            __threadfence();
            __syncwarp();
            int prior = 0;
            if (lane == 0) prior = atomicAdd(p.arrivals + tree_first[k], 1);
            prior = __shfl_sync(0xffffffffu, prior, 0);
            if (prior != n_grp[k] - 1) continue;
            __threadfence();
            if (lane == 0) p.arrivals[tree_first[k]] = 0;
            jobs[n_jobs] = grid_job(tree_first[k], n_grp[k], 0, sub[k], -1, 0u, false);
            jobs[n_jobs].out_rows = tree_out[k];
            ++n_jobs;
        }
    }

    // ---- run the grid-stage jobs.  The rounds of a fold (and with them its rounding) must not depend
    // on which warp happened to come last, so a job's round size is a function of its own size only:
    // two jobs that each fit half the ring in one round share it, their fetches in flight together;
    // otherwise a job has the whole ring and the second one starts after the first.
    if (alive && n_jobs > 0) {
        const int whole = NS * Lay::kStageBytes;
        const bool share = n_jobs == 2 && max(jobs[0].n, jobs[1].n) <= (whole / 2) / part_bytes;
#pragma unroll 1
        for (int s = 0; s < 2 * n_jobs && alive; ++s) {
            const int i = share ? (s & 1) : (s >> 1);
            const bool fetch = share ? s < 2 : !(s & 1);
            if (fetch) {
                jobs[i].base = ring + 64 + (share ? i * (whole / 2) : 0);
                jobs[i].cap = min(32, (share ? whole / 2 : whole) / part_bytes);
                jobs[i].bar = bars + i * 8;
                jobs[i].uses = bar_uses[i];
                fence_proxy_async();              // generic-proxy accesses (the partials' stores, an earlier job's reads) before the copies
                __syncwarp();
                fold_fetch<D>(jobs[i], fc, 0);
            } else if (fold_finish<D>(jobs[i], fc) < 0) {
                alive = false;
            }
        }
    }

    // Do not leave while copies into this warp's ring may still be in flight (only after a wait gave up).
    if (!alive) {
        for (int k = landed; k < issued; ++k) mbar_wait_bounded(bars + (k % NS) * 8, (k / NS) & 1, p.status);
    }
    if (lane == 0) {
        p.trace[span * 8 + 3] = global_timer_ns();
        p.trace[span * 8 + 4] = t_wait;
#ifdef CKV_TRACE_WAITS
        p.trace[span * 8 + 5] = t_between;
#else
        { unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); p.trace[span * 8 + 5] = smid; }
#endif
#ifdef CKV_TRACE_WAITS
        p.trace[span * 8 + 6] = t_issue;
        p.trace[span * 8 + 7] = t_masked;
#else
        p.trace[span * 8 + 6] = done;
        p.trace[span * 8 + 7] = n_pieces;
#endif
    }
}

// ------------------------------------------------------------------------------------------
// Self-test of the give-up path of the bounded waits.  One warp waits, with the same routine the
// attention kernel uses but a caller-given limit, for a phase of an mbarrier that nothing will ever
// complete: no copy is issued and nobody arrives.  When the limit runs out the routine flags the
// status word and returns, and the warp leaves an arrival counter half-way, as an attention warp
// that gave up in the middle of a merge would.  Nothing here can fault or hang: the only loop is
// the bounded one.
// ------------------------------------------------------------------------------------------
__global__ void wait_limit_selftest_kernel(uint32_t *status, int32_t *arrivals, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    bool ok = mbar_wait_bounded(bar, 0, status, limit_ns);      // phase 0 never completes
    ok = __all_sync(0xffffffffu, ok);
    if (!ok && threadIdx.x == 0) atomicAdd(arrivals, 1);
}

// ------------------------------------------------------------------------------------------
// Read probe: the attention kernel's loads without its arithmetic.  Every warp takes the same span
// of the same plan, fetches the same tiles with the same TMA boxes through a ring of the same
// depth, and only waits for them to land.  What this kernel takes is what the memory system gives
// this access pattern: the practical ceiling the attention kernel is measured against.
// ------------------------------------------------------------------------------------------
struct ProbeParams {
    const int32_t *block_tables;
    const int32_t *seq_lens;
    uint32_t *status;
    unsigned long long *sink;       // receives a checksum of a few loaded words so that the loads count
    int32_t batch, max_pages_per_req, num_pages, num_kv_heads;
    int32_t layer_page_base, num_spans;
};

template <int D, int W, int NS>
__global__ void __launch_bounds__(W * 32, 1)
pool_read_probe_kernel(const __grid_constant__ CUtensorMap tmap, const ProbeParams p)
{
    using Lay = AttnLayout<D, W, NS>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int span = blockIdx.x * W + warp;
    if (span >= p.num_spans) return;
    const uint32_t ring = smem_u32(smem) + warp * NS * Lay::kStageBytes;
    const uint32_t bars = smem_u32(smem + Lay::kBarOff) + warp * NS * 8;
    if (lane == 0) {
        prefetch_tensormap(&tmap);
        for (int s = 0; s < NS; ++s) mbar_init(bars + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncwarp();
    const SpanStart st = warp_plan(p.seq_lens, p.batch, p.max_pages_per_req, p.num_kv_heads, p.num_spans, span, lane);
    if (st.r < 0) return;
    AttnParams ap{};                              // the cursor reads only these
    ap.seq_lens = p.seq_lens; ap.batch = p.batch; ap.max_pages_per_req = p.max_pages_per_req;
    ap.num_kv_heads = p.num_kv_heads; ap.q_len = 1;
    const uint64_t policy = l2_evict_first_policy();
    SpanCursor ic;
    ic.r = st.r; ic.h = st.h; ic.tile = st.tile; ic.L = st.L; ic.tiles = st.tiles_r; ic.v = st.v;
    bool more = true;
    int issued = 0, done = 0;
    auto issue = [&]() {
        const int n_pages = (ic.L + kPageSize - 1) / kPageSize;
        const int np = min(kPagesPerTile, n_pages - ic.tile * kPagesPerTile);
        const int pg = lane / Lay::kHalves, hf = lane % Lay::kHalves;
        const int slot = issued % NS;
        if (lane == 0) mbar_arrive_expect_tx(bars + slot * 8, np * Lay::kPageBytes);
        __syncwarp();
        if (lane < np * Lay::kHalves) {
            int page = __ldg(p.block_tables + (size_t)ic.r * p.max_pages_per_req + ic.tile * kPagesPerTile + pg);
            if (page < 0 || page >= p.num_pages) { atomicOr(p.status, kStatusBadPage); page = 0; }
            const int y = ((p.layer_page_base + page) * p.num_kv_heads + ic.h) * 32;
            tma_load_2d(ring + slot * Lay::kStageBytes + pg * Lay::kPageBytes + hf * Lay::kHalfBytes, &tmap, hf * 64, y,
                        bars + slot * 8, policy);
        }
        ++issued;
        more = ic.next(ap) && ic.v < st.end;
    };
    for (int k = 0; k < NS && more; ++k) issue();
    uint32_t acc = 0;
    bool alive = true;
    while (done < issued) {
        // every copy issued is waited for (each wait bounded), also after one of them gave up
        const bool ok = mbar_wait_bounded(bars + (done % NS) * 8, (done / NS) & 1, p.status);
        if (!__all_sync(0xffffffffu, ok)) alive = false;
        if (alive) {
            uint32_t v;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(ring + (done % NS) * Lay::kStageBytes + lane * 4));
            acc ^= v;
        }
        ++done;
        if (more && alive) issue();
    }
    if (acc == 0x9e3779b9u && lane == 0) atomicAdd(p.sink, 1ull);     // keeps the loads alive; practically never taken
}

}  // namespace ckv
