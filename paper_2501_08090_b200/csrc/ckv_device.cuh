// Device code of the decode-iteration hot path for sm_100a: KV append, split-KV plan,
// paged grouped-query partial attention (TMA-fed, tensor-core) and the log-sum-exp combine.
//
// Pool layout (bf16): [layer][page][kv_head][K|V][slot 0..15][d]  -- one (page, kv_head) is a
// contiguous block of 32 rows (16 key rows, then 16 value rows) of d elements.
#pragma once

#include <cuda.h>            // CUtensorMap (type only; the driver library is not linked)
#include <cuda_runtime.h>
#include <stdint.h>

namespace ckv {

constexpr int kPageSize = 16;        // tokens per page
constexpr int kPagesPerTile = 4;     // a tile is the scheduling unit: 64 tokens of one (request, kv head)
constexpr int kTileTokens = kPageSize * kPagesPerTile;
constexpr int kMaxGroup = 8;         // query heads per KV head handled by one MMA column block
constexpr int kMaxCtas = 1024;       // upper bound on the partition width
constexpr int kMaxBatch = 8192;

constexpr uint32_t kStatusBadLength = 1u;
constexpr uint32_t kStatusBadPage = 2u;
constexpr uint32_t kStatusWaitLimit = 4u;

constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // bound of every device-side wait

struct PlanHeader {
    int32_t total_tiles;      // over all (request, kv head)
    int32_t tiles_per_cta;    // span length q: CTA c owns tiles [c*q, min((c+1)*q, total))
    int32_t num_ctas;         // partition width
    int32_t ctas_with_work;
};

// A context length is usable if 1 <= L <= table capacity; otherwise the request has no tiles.
__host__ __device__ __forceinline__ int tiles_of_length(int L, int max_pages_per_req)
{
    if (L < 1 || (long long)L > (long long)max_pages_per_req * kPageSize) return 0;
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
};

__global__ void kv_append_kernel(const AppendParams p)
{
    const int vec_per_row = p.head_dim / 8;                       // 16-byte pieces per row
    const int per_req = p.num_kv_heads * 2 * vec_per_row;
    const long long total = (long long)p.batch * per_req;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(idx / per_req);
        int rem = (int)(idx % per_req);
        const int kh = rem / (2 * vec_per_row);
        rem -= kh * 2 * vec_per_row;
        const int kv = rem / vec_per_row;
        const int c = rem % vec_per_row;

        const int L = p.seq_lens[r];
        if (tiles_of_length(L, p.max_pages_per_req) == 0) {
            if (rem == 0 && kh == 0) atomicOr(p.status, kStatusBadLength);
            continue;
        }
        const int pos = L - 1;
        const int page = p.block_tables[(size_t)r * p.max_pages_per_req + pos / kPageSize];
        if (page < 0 || page >= p.num_pages) {
            if (rem == 0 && kh == 0) atomicOr(p.status, kStatusBadPage);
            continue;
        }
        const int slot = pos % kPageSize;
        const uint4 *src = (kv == 0 ? p.k_new : p.v_new) + ((size_t)r * p.num_kv_heads + kh) * vec_per_row + c;
        const size_t row = (((size_t)page * p.num_kv_heads + kh) * 2 + kv) * kPageSize + slot;
        p.pool_layer[row * vec_per_row + c] = *src;
    }
}

// ------------------------------------------------------------------------------------------
// K2: split-KV plan.  One CTA: per-request tile counts, their exclusive prefix sum, the span
// length, and for every CTA of the partition the (request, kv head, tile) its span starts at.
// ------------------------------------------------------------------------------------------
struct PlanParams {
    const int32_t *seq_lens;
    PlanHeader *header;
    int4 *cta_start;                // [num_ctas]
    int32_t *tile_prefix;           // [batch + 1], tiles per KV head before request r
    uint32_t *status;
    uint16_t *out;                  // rows of requests with an unusable length are zero-filled
    int32_t batch, max_pages_per_req, num_kv_heads, num_ctas, out_row_elems;
};

constexpr int kPlanThreads = 1024;

__global__ void __launch_bounds__(kPlanThreads) splitkv_plan_kernel(const PlanParams p)
{
    extern __shared__ int32_t s_prefix[];        // [batch + 1]
    __shared__ int32_t s_warp[32];
    const int tid = threadIdx.x;
    const int per = (p.batch + kPlanThreads - 1) / kPlanThreads;
    const int r0 = tid * per;
    const int r1 = min(p.batch, r0 + per);

    int local = 0;
    for (int r = r0; r < r1; ++r) {
        const int t = tiles_of_length(p.seq_lens[r], p.max_pages_per_req);
        if (t == 0) {
            atomicOr(p.status, kStatusBadLength);
            if (p.out != nullptr)
                for (int i = 0; i < p.out_row_elems; ++i) p.out[(size_t)r * p.out_row_elems + i] = 0;
        }
        s_prefix[r] = t;                          // overwritten by the prefix below
        local += t;
    }
    // exclusive scan of the per-thread sums
    int incl = local;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = s_warp[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += v;
        }
        s_warp[lane] = w;                         // inclusive over warps
    }
    __syncthreads();
    int run = incl - local + (warp > 0 ? s_warp[warp - 1] : 0);
    for (int r = r0; r < r1; ++r) {
        const int t = s_prefix[r];
        s_prefix[r] = run;
        run += t;
    }
    if (tid == kPlanThreads - 1) s_prefix[p.batch] = s_warp[31];
    __syncthreads();

    const int per_head_total = s_prefix[p.batch];
    const int total = per_head_total * p.num_kv_heads;
    const int q = max(1, (total + p.num_ctas - 1) / p.num_ctas);
    for (int r = tid; r <= p.batch; r += kPlanThreads) p.tile_prefix[r] = s_prefix[r];
    if (tid == 0) {
        p.header->total_tiles = total;
        p.header->tiles_per_cta = q;
        p.header->num_ctas = p.num_ctas;
        p.header->ctas_with_work = (total + q - 1) / q;
    }
    for (int c = tid; c < p.num_ctas; c += kPlanThreads) {
        const long long t0 = (long long)c * q;
        int4 st = make_int4(-1, -1, -1, -1);
        if (t0 < total) {
            // smallest r' with Hkv*prefix[r'] > t0; the span starts inside request r' - 1
            int lo = 0, hi = p.batch;             // prefix[0] = 0 <= t0 < Hkv*prefix[batch]
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if ((long long)s_prefix[mid] * p.num_kv_heads > t0) hi = mid; else lo = mid;
            }
            const int r = lo;
            const int tr = s_prefix[r + 1] - s_prefix[r];
            const int rem = (int)(t0 - (long long)s_prefix[r] * p.num_kv_heads);
            st = make_int4(r, rem / tr, rem % tr, (int)t0);
        }
        p.cta_start[c] = st;
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

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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

// Wait for a phase of an mbarrier, giving up after kWaitLimitNs or as soon as another thread of
// the CTA has given up.  Returns false when it gave up (the caller then skips its work).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                                  uint32_t *status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > kWaitLimitNs) {
            *abort_flag = 1;
            atomicOr(status, kStatusWaitLimit);
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
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

__device__ __forceinline__ void named_barrier_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ uint16_t f32_to_bf16_rn(float x)
{
    uint16_t h;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(x));
    return h;
}

// ------------------------------------------------------------------------------------------
// K3: paged partial attention.
//
// One persistent CTA per span of the plan.  Warp W (the last) is the producer: it walks the
// span tile by tile, looks the pages up in the block table and issues one TMA box load per
// 128-byte column block of each (page, kv head) into a ring of S stages (one stage = one tile =
// up to 4 pages).  Warps 0..W-1 are consumers; stage number `it` of the CTA is consumed by warp
// it % W, which keeps its own running maximum m, sum l and accumulator O for the current
// (request, kv head) piece.  At the end of a piece the consumer warps merge their states through
// shared memory and write either the final bf16 output row (the piece covered the whole
// context) or an fp32 partial (m, l, O) for the combine kernel.
//
// MMA formulation (operands swapped so the tile's tokens fill the M dimension):
//   S^T[tok 16 x g 8]  = K[tok 16 x d] . Q^T[d x g 8]          (A = K rows via ldmatrix)
//   O^T[d 16 x g 8]   += V^T[d 16 x tok 16] . P^T[tok 16 x g 8] (A = V via ldmatrix.trans)
// The S^T accumulator fragment holds (token = lane/4 [+8], g = 2*(lane%4)+{0,1}); packed to bf16
// and transposed with movmatrix it is exactly the B fragment of P^T.
// ------------------------------------------------------------------------------------------
struct AttnParams {
    const int32_t *block_tables;
    const int32_t *seq_lens;
    const uint16_t *q;
    uint16_t *out;
    const PlanHeader *header;
    const int4 *cta_start;
    float *part_acc;                // [2*kMaxCtas][8][D]
    float *part_ml;                 // [2*kMaxCtas][16]  (m[8], l[8])
    uint32_t *status;
    unsigned long long *cta_trace;  // [gridDim.x][4] ns: CTA start, first data consumed, producer done, consumers done
    int32_t batch, max_pages_per_req, num_pages, num_kv_heads, num_q_heads, group;
    int32_t layer_page_base;        // layer * num_pages
    float scale_log2;               // log2(e) / sqrt(d)
};

template <int D, int W, int S>
struct AttnLayout {
    static constexpr int kHalves = D / 64;                       // 128-byte column blocks per row
    static constexpr int kHalfBytes = 32 * 128;                  // one TMA box: 32 rows x 128 B
    static constexpr int kPageBytes = kHalves * kHalfBytes;      // K and V rows of one (page, head)
    static constexpr int kStageBytes = kPagesPerTile * kPageBytes;
    static constexpr int kKSteps = D / 16;
    static constexpr int kDTiles = D / 16;
    static constexpr int kScratchFloats = W * D * kMaxGroup + W * 2 * kMaxGroup;
    static constexpr int kSmemBytes = S * kStageBytes + kScratchFloats * 4 + 2 * S * 8 + 16 + 1024;
    static constexpr int kThreads = (W + 1) * 32;
};

// Position of a CTA inside its span; producer and consumers advance identical copies.
struct SpanWalk {
    int r, h, tile;       // next tile to process: request, kv head, tile within (r, h)
    int remaining;        // tiles left in the span
    int L, tiles;         // length and tile count of request r

    __device__ __forceinline__ void load_request(const AttnParams &p)
    {
        L = p.seq_lens[r];
        tiles = tiles_of_length(L, p.max_pages_per_req);
    }
    // tiles of the current piece
    __device__ __forceinline__ int piece_tiles() const { return min(tiles - tile, remaining); }
    // move past the current piece to the start of the next (request, kv head)
    __device__ __forceinline__ void advance(const AttnParams &p, int n)
    {
        remaining -= n;
        if (remaining <= 0) return;
        tile = 0;
        if (++h == p.num_kv_heads) {
            h = 0;
            do {
                if (++r >= p.batch) { remaining = 0; return; }
                load_request(p);
            } while (tiles == 0);
        }
    }
};

template <int D, int W, int S>
__global__ void __launch_bounds__((W + 1) * 32, 1)
paged_decode_attn_kernel(const __grid_constant__ CUtensorMap tmap, const AttnParams p)
{
    using Lay = AttnLayout<D, W, S>;
    // Stage `it` lives in slot it % S and is consumed by warp it % W.  A consumer tells "my data
    // has landed" from the parity of the slot's barrier, which is only unambiguous if it cannot
    // get a whole phase ahead of the slot's previous use.  Copies complete out of order, so that
    // holds only when the previous use of the slot was consumed by the SAME warp: S % W == 0.
    static_assert(S % W == 0, "every ring slot must always be consumed by the same warp");
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float *scratch_o = (float *)(smem + S * Lay::kStageBytes);            // [W][D][8]
    float *scratch_ml = scratch_o + W * D * kMaxGroup;                     // [W][16]
    uint64_t *bars = (uint64_t *)(scratch_ml + W * 2 * kMaxGroup);         // full[S], empty[S]
    volatile int *abort_flag = (volatile int *)(bars + 2 * S);

    const uint32_t stage_base = smem_u32(smem);
    const uint32_t full_bar = smem_u32(bars);
    const uint32_t empty_bar = full_bar + S * 8;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_bar + s * 8, 1);
            mbar_init(empty_bar + s * 8, 1);
        }
        *abort_flag = 0;
        p.cta_trace[blockIdx.x * 4 + 0] = global_timer_ns();
        p.cta_trace[blockIdx.x * 4 + 1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int total = p.header->total_tiles;
    const int q_span = p.header->tiles_per_cta;
    const long long span_begin = (long long)blockIdx.x * q_span;
    if (span_begin >= total) return;
    const int4 st = p.cta_start[blockIdx.x];

    SpanWalk wk;
    wk.r = st.x; wk.h = st.y; wk.tile = st.z;
    wk.remaining = (int)min((long long)q_span, (long long)total - span_begin);
    wk.load_request(p);

    if (warp == W) {
        // ------------------------------------------------------------------ producer warp
        int it = 0;
        bool ok = true;
        int pf_val = -1, pf_row = -1;              // chunk 0 of the row the next piece is expected in
        while (wk.remaining > 0 && ok) {
            const int n = wk.piece_tiles();
            const int n_pages = (wk.L + kPageSize - 1) / kPageSize;
            const int32_t *row = p.block_tables + (size_t)wk.r * p.max_pages_per_req;
            auto load_chunk = [&](const int32_t *rw, int chunk) -> int {
                const int idx = chunk * 32 + lane;
                return idx < p.max_pages_per_req ? __ldg(rw + idx) : -1;
            };
            int cur_chunk = wk.tile / 8;
            int cur_val = (cur_chunk == 0 && pf_row == wk.r) ? pf_val : load_chunk(row, cur_chunk);
            int nxt_val = load_chunk(row, cur_chunk + 1);
            // the next piece starts at tile 0 of this row (next kv head) or of the next request
            pf_row = (wk.h + 1 < p.num_kv_heads) ? wk.r : wk.r + 1;
            pf_val = (pf_row < p.batch) ? load_chunk(p.block_tables + (size_t)pf_row * p.max_pages_per_req, 0) : -1;

            for (int ti = wk.tile; ti < wk.tile + n && ok; ++ti, ++it) {
                const int ck = ti / 8;
                if (ck != cur_chunk) {
                    cur_chunk = ck;
                    cur_val = nxt_val;
                    nxt_val = load_chunk(row, ck + 1);
                }
                const int np = min(kPagesPerTile, n_pages - ti * kPagesPerTile);
                const int pg = lane / Lay::kHalves, hf = lane % Lay::kHalves;
                int page = __shfl_sync(0xffffffffu, cur_val, ((ti & 7) * kPagesPerTile + pg) & 31);
                const int slot = it % S;
                ok = mbar_wait_bounded(empty_bar + slot * 8, ((it / S) & 1) ^ 1, abort_flag, p.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane == 0) mbar_arrive_expect_tx(full_bar + slot * 8, np * Lay::kPageBytes);
                __syncwarp();
                if (lane < np * Lay::kHalves) {
                    if (page < 0 || page >= p.num_pages) {
                        atomicOr(p.status, kStatusBadPage);
                        page = 0;
                    }
                    const int y = ((p.layer_page_base + page) * p.num_kv_heads + wk.h) * 32;
                    tma_load_2d(stage_base + slot * Lay::kStageBytes + pg * Lay::kPageBytes + hf * Lay::kHalfBytes,
                                &tmap, hf * 64, y, full_bar + slot * 8);
                }
            }
            wk.advance(p, n);
        }
        // Do not leave the CTA while copies into its shared memory may still be in flight.
        if (lane == 0) {
            p.cta_trace[blockIdx.x * 4 + 2] = global_timer_ns();
            for (int k = max(0, it - S); k < it; ++k) {
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(full_bar + (k % S) * 8, (k / S) & 1)) {
                    if (global_timer_ns() - t0 > kWaitLimitNs) {
                        atomicOr(p.status, kStatusWaitLimit);
                        break;
                    }
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    const int g_row = lane >> 2;                 // query head (within the group) this lane loads Q for
    const int g0 = (lane & 3) * 2;               // first of the two group columns this lane accumulates
    const int G = p.group;

    // ldmatrix lane offsets inside one page block (without the column-block and page terms)
    uint32_t k_off[4], v_off[4];
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

    int it = 0;
    bool alive = true;
    bool first_piece = true;
    while (wk.remaining > 0) {
        const int n = wk.piece_tiles();
        const bool complete = (wk.tile == 0 && n == wk.tiles);

        // Q^T fragments of this (request, kv head): b0/b1 of k-step ks hold
        // Q[g_row][ks*16 + 2*(lane%4) + {0,1}] and the same columns + 8.
        uint32_t qf[Lay::kKSteps][2];
        {
            const uint32_t *qrow = (const uint32_t *)(p.q + ((size_t)wk.r * p.num_q_heads + wk.h * G + g_row) * D);
#pragma unroll
            for (int ks = 0; ks < Lay::kKSteps; ++ks) {
                qf[ks][0] = g_row < G ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
                qf[ks][1] = g_row < G ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
            }
        }
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[Lay::kDTiles][4];
#pragma unroll
        for (int dt = 0; dt < Lay::kDTiles; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;

        for (int ti = wk.tile; ti < wk.tile + n; ++ti, ++it) {
            if (it % W != warp) continue;
            const int slot = it % S;
            if (alive) {
                alive = mbar_wait_bounded(full_bar + slot * 8, (it / S) & 1, abort_flag, p.status);
                alive = __all_sync(0xffffffffu, alive);
            }
            if (!alive) continue;
            if (it == 0 && lane == 0) p.cta_trace[blockIdx.x * 4 + 1] = global_timer_ns();

            const int ntok = min(kTileTokens, wk.L - ti * kTileTokens);     // valid tokens in this tile
            const bool full_tile = (ntok == kTileTokens);
            const int np = (ntok + kPageSize - 1) / kPageSize;
            const uint32_t sb = stage_base + slot * Lay::kStageBytes;

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
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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

            // ---- online softmax in the log2 domain
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int mt = 0; mt < kPagesPerTile; ++mt) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tok = mt * kPageSize + (lane >> 2) + (i >= 2 ? 8 : 0);
                    const float t = (full_tile || tok < ntok) ? s[mt][i] * p.scale_log2 : -INFINITY;
                    s[mt][i] = t;
                    if (i & 1) mx1 = fmaxf(mx1, t); else mx0 = fmaxf(mx0, t);
                }
            }
#pragma unroll
            for (int x = 4; x < 32; x <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, x));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, x));
            }
            const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
            const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);
            m0 = mn0; m1 = mn1;
            l0 *= al0; l1 *= al1;
#pragma unroll
            for (int dt = 0; dt < Lay::kDTiles; ++dt) {
                o[dt][0] *= al0; o[dt][2] *= al0;
                o[dt][1] *= al1; o[dt][3] *= al1;
            }
            uint32_t pb[kPagesPerTile][2];
#pragma unroll
            for (int mt = 0; mt < kPagesPerTile; ++mt) {
                const float p0 = fast_exp2(s[mt][0] - mn0), p1 = fast_exp2(s[mt][1] - mn1);
                const float p2 = fast_exp2(s[mt][2] - mn0), p3 = fast_exp2(s[mt][3] - mn1);
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
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar + slot * 8);
        }

        // ---- merge the W warps' states of this piece and write it out
#pragma unroll
        for (int x = 4; x < 32; x <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, x);
            l1 += __shfl_xor_sync(0xffffffffu, l1, x);
        }
        {
            float *so = scratch_o + (size_t)warp * D * kMaxGroup;
#pragma unroll
            for (int dt = 0; dt < Lay::kDTiles; ++dt) {
                const int d = dt * 16 + (lane >> 2);
                *(float2 *)(so + d * kMaxGroup + g0) = make_float2(o[dt][0], o[dt][1]);
                *(float2 *)(so + (d + 8) * kMaxGroup + g0) = make_float2(o[dt][2], o[dt][3]);
            }
            if (lane < 4) {
                float *ml = scratch_ml + warp * 2 * kMaxGroup;
                ml[g0] = m0; ml[g0 + 1] = m1;
                ml[kMaxGroup + g0] = l0; ml[kMaxGroup + g0 + 1] = l1;
            }
        }
        named_barrier_sync(1, W * 32);
        {
            float f[W][kMaxGroup], mstar[kMaxGroup], lsum[kMaxGroup];
#pragma unroll
            for (int g = 0; g < kMaxGroup; ++g) {
                float mm = -INFINITY;
#pragma unroll
                for (int w = 0; w < W; ++w) mm = fmaxf(mm, scratch_ml[w * 2 * kMaxGroup + g]);
                mstar[g] = mm;
                float ls = 0.f;
#pragma unroll
                for (int w = 0; w < W; ++w) {
                    f[w][g] = fast_exp2(scratch_ml[w * 2 * kMaxGroup + g] - mm);   // idle warp: exp2(-inf) = 0
                    ls += f[w][g] * scratch_ml[w * 2 * kMaxGroup + kMaxGroup + g];
                }
                lsum[g] = ls;
            }
            const int slot_id = 2 * blockIdx.x + (first_piece ? 0 : 1);
            for (int d = threadIdx.x; d < D; d += W * 32) {
                float acc[kMaxGroup];
#pragma unroll
                for (int g = 0; g < kMaxGroup; ++g) acc[g] = 0.f;
#pragma unroll
                for (int w = 0; w < W; ++w) {
                    const float4 a = *(const float4 *)(scratch_o + ((size_t)w * D + d) * kMaxGroup);
                    const float4 b = *(const float4 *)(scratch_o + ((size_t)w * D + d) * kMaxGroup + 4);
                    acc[0] += f[w][0] * a.x; acc[1] += f[w][1] * a.y; acc[2] += f[w][2] * a.z; acc[3] += f[w][3] * a.w;
                    acc[4] += f[w][4] * b.x; acc[5] += f[w][5] * b.y; acc[6] += f[w][6] * b.z; acc[7] += f[w][7] * b.w;
                }
                if (complete) {
#pragma unroll
                    for (int g = 0; g < kMaxGroup; ++g)
                        if (g < G)
                            p.out[((size_t)wk.r * p.num_q_heads + wk.h * G + g) * D + d] = f32_to_bf16_rn(acc[g] / lsum[g]);
                } else {
#pragma unroll
                    for (int g = 0; g < kMaxGroup; ++g)
                        p.part_acc[((size_t)slot_id * kMaxGroup + g) * D + d] = acc[g];
                }
            }
            if (!complete && threadIdx.x < kMaxGroup) {
                p.part_ml[slot_id * 2 * kMaxGroup + threadIdx.x] = mstar[threadIdx.x];
                p.part_ml[slot_id * 2 * kMaxGroup + kMaxGroup + threadIdx.x] = lsum[threadIdx.x];
            }
        }
        named_barrier_sync(1, W * 32);            // scratch is reused by the next piece
        first_piece = false;
        wk.advance(p, n);
    }
    if (threadIdx.x == 0) p.cta_trace[blockIdx.x * 4 + 3] = global_timer_ns();
}

// ------------------------------------------------------------------------------------------
// K4: log-sum-exp combine.  Block c looks at the boundary between spans c and c+1.  If that
// boundary cuts a (request, kv head) and is the first one to cut it, the block merges all the
// partials of that (request, kv head) and writes its bf16 output rows.
// ------------------------------------------------------------------------------------------
struct CombineParams {
    const PlanHeader *header;
    const int32_t *tile_prefix;
    const float *part_acc;
    const float *part_ml;
    uint16_t *out;
    int32_t batch, num_kv_heads, num_q_heads, group, head_dim;
};

__global__ void lse_combine_kernel(const CombineParams p)
{
    const int total = p.header->total_tiles;
    const int q = p.header->tiles_per_cta;
    const int c = blockIdx.x;
    const long long tb = (long long)(c + 1) * q;            // first tile of span c + 1
    if (tb >= total) return;

    // (request, kv head) containing tile tb
    int lo = 0, hi = p.batch;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)p.tile_prefix[mid] * p.num_kv_heads > tb) hi = mid; else lo = mid;
    }
    const int r = lo;
    const int tr = p.tile_prefix[r + 1] - p.tile_prefix[r];
    const int rem = (int)(tb - (long long)p.tile_prefix[r] * p.num_kv_heads);
    const int h = rem / tr, tile = rem % tr;
    if (tile == 0) return;                                  // boundary falls between two pieces
    const long long item_begin = tb - tile, item_end = item_begin + tr;
    if ((long long)c * q > item_begin) return;              // an earlier boundary already cuts it

    const int first_slot = ((long long)c * q == item_begin) ? 2 * c : 2 * c + 1;
    int last_cta = c + 1;
    while ((long long)(last_cta + 1) * q < item_end) ++last_cta;
    const int pieces = last_cta - c + 1;

    const int D = p.head_dim, G = p.group;
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int g = idx / D, d = idx % D;
        float mstar = -INFINITY;
        for (int i = 0; i < pieces; ++i) {
            const int slot = (i == 0) ? first_slot : 2 * (c + i);
            mstar = fmaxf(mstar, p.part_ml[slot * 2 * kMaxGroup + g]);
        }
        float lsum = 0.f, acc = 0.f;
        for (int i = 0; i < pieces; ++i) {
            const int slot = (i == 0) ? first_slot : 2 * (c + i);
            const float f = fast_exp2(p.part_ml[slot * 2 * kMaxGroup + g] - mstar);
            lsum += f * p.part_ml[slot * 2 * kMaxGroup + kMaxGroup + g];
            acc += f * p.part_acc[((size_t)slot * kMaxGroup + g) * D + d];
        }
        p.out[((size_t)r * p.num_q_heads + h * G + g) * D + d] = f32_to_bf16_rn(acc / lsum);
    }
}

}  // namespace ckv
