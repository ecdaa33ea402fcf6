// Host runtime and C ABI (include/chiron_kv.h) of the paged decode-attention library.
// Argument checking, workspace carving, tensor-map creation, kernel launches and timing loops.
// No device memory is allocated here: pool and workspace belong to the caller.
#include "chiron_kv.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "ckv_device.cuh"

namespace {

thread_local char g_error[512] = "";

int32_t fail(int32_t code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
    return code;
}

#define CKV_CUDA(call)                                                                        \
    do {                                                                                      \
        cudaError_t e_ = (call);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return fail(CKV_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_),    \
                        __FILE__, __LINE__);                                                  \
    } while (0)

// Attention kernel shapes: warps per CTA (one CTA per SM) and ring stages per warp.
#ifndef CKV_WARPS128
#define CKV_WARPS128 4
#endif
#ifndef CKV_STAGES128
#define CKV_STAGES128 3
#endif
#ifndef CKV_WARPS64
#define CKV_WARPS64 4
#endif
#ifndef CKV_STAGES64
#define CKV_STAGES64 4
#endif
constexpr int kWarps128 = CKV_WARPS128, kStages128 = CKV_STAGES128;   // head_dim 128: 4 warps x 3 stages x 16 KB = 192 KB per SM
constexpr int kWarps64 = CKV_WARPS64, kStages64 = CKV_STAGES64;       // head_dim 64:  4 warps x 4 stages x 8 KB
constexpr int kMaxProfile = 4096;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool config_ok(const ckv_config *c, const char **why)
{
    *why = "";
    if (!c) { *why = "config is NULL"; return false; }
    if (c->num_layers < 1) { *why = "num_layers < 1"; return false; }
    if (c->head_dim != 64 && c->head_dim != 128) { *why = "head_dim must be 64 or 128"; return false; }
    if (c->page_size != ckv::kPageSize) { *why = "page_size must be 16"; return false; }
    if (c->num_kv_heads < 1 || c->num_q_heads < 1 || c->num_q_heads % c->num_kv_heads != 0) {
        *why = "num_q_heads must be a positive multiple of num_kv_heads"; return false;
    }
    if (c->num_q_heads / c->num_kv_heads > ckv::kMaxGroup) { *why = "group size above 8"; return false; }
    if (c->num_pages < 1) { *why = "num_pages < 1"; return false; }
    if (c->max_pages_per_req < 1) { *why = "max_pages_per_req < 1"; return false; }
    if (c->max_batch < 1 || c->max_batch > ckv::kMaxBatch) { *why = "max_batch outside [1, 8192]"; return false; }
    // TMA row coordinates are int32
    const long long rows = (long long)c->num_layers * c->num_pages * c->num_kv_heads * 32;
    if (rows >= (1ll << 31)) { *why = "pool has 2^31 or more rows"; return false; }
    // tile counts are int32
    const long long tiles = (long long)c->max_batch * c->num_kv_heads *
                            (((long long)c->max_pages_per_req * ckv::kPageSize + ckv::kTileTokens - 1) / ckv::kTileTokens);
    if (tiles >= (1ll << 31)) { *why = "max_batch * max context has 2^31 or more tiles"; return false; }
    return true;
}

struct WorkspaceLayout {
    size_t status, header, span_start, part, arrivals, trace;
    size_t st_tables, st_lens, st_q, st_k, st_v, st_out;
    size_t total;
};

WorkspaceLayout carve(const ckv_config &c)
{
    WorkspaceLayout w{};
    size_t at = 0;
    auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes, 256); return o; };
    const size_t d2 = (size_t)c.head_dim * 2;
    w.status = take(256);
    w.header = take(sizeof(ckv::PlanHeader));
    w.span_start = take(sizeof(int4) * ckv::kMaxSpans);
    w.part = take(sizeof(float) * 2 * ckv::kMaxSpans * (2 * ckv::kMaxGroup + ckv::kMaxGroup * c.head_dim));
    w.arrivals = take(sizeof(int32_t) * ckv::kMaxSpans);
    w.trace = take(sizeof(unsigned long long) * 8 * ckv::kMaxSpans);
    w.st_tables = take(sizeof(int32_t) * (size_t)c.max_batch * c.max_pages_per_req);
    w.st_lens = take(sizeof(int32_t) * (size_t)c.max_batch);
    w.st_q = take((size_t)c.max_batch * c.num_q_heads * d2);
    w.st_k = take((size_t)c.max_batch * c.num_kv_heads * d2);
    w.st_v = take((size_t)c.max_batch * c.num_kv_heads * d2);
    w.st_out = take((size_t)c.max_batch * c.num_q_heads * d2);
    w.total = at;
    return w;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled, looked up once per process (the driver library is not linked).
EncodeTiledFn encode_tiled_fn(const char **why)
{
    static EncodeTiledFn cached = nullptr;
    if (cached) return cached;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        *why = cudaGetErrorString(e);
        return nullptr;
    }
    cached = reinterpret_cast<EncodeTiledFn>(fn);
    return cached;
}

// Tensor map over a whole pool seen as rows of head_dim bf16; one box = 32 rows (the 16 key rows
// and 16 value rows of one (page, kv head)) x 64 columns, stored with the 128-byte swizzle.
int32_t encode_pool_map(const ckv_config *cfg, const void *d_pool, CUtensorMap *out, const char *fn_name)
{
    const char *why = "";
    const EncodeTiledFn encode = encode_tiled_fn(&why);
    if (!encode) return fail(CKV_ECUDA, "%s: cuTensorMapEncodeTiled not available (%s)", fn_name, why);
    const cuuint64_t rows = (cuuint64_t)cfg->num_layers * cfg->num_pages * cfg->num_kv_heads * 32;
    const cuuint64_t dims[2] = {(cuuint64_t)cfg->head_dim, rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cfg->head_dim * 2};
    const cuuint32_t box[2] = {64, 32};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult cr = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(d_pool), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(CKV_ECUDA, "%s: cuTensorMapEncodeTiled returned %d", fn_name, (int)cr);
    return CKV_OK;
}

}  // namespace

struct ckv_pool {
    ckv_config cfg;
    int device;
    int num_sms;
    int num_spans;                   // partition width: one span per warp of the attention kernel
    uint8_t *d_pool;
    uint8_t *d_ws;
    WorkspaceLayout ws;
    CUtensorMap tmap;
    int64_t launches;
    bool profile;
    bool overlap;                    // launch kernels with programmatic stream serialization
    bool pool_written;               // a kernel other than the fused step wrote the pool since the last attention launch
    bool inputs_from_predecessor;    // the next attention launch reads tables and lengths its predecessor in the stream writes
    int host_route;                  // decode_step_host: CKV_HOST_ROUTE_*
    std::vector<cudaEvent_t> ev;     // pairs (start, stop)
    int ev_used;

    template <typename T> T *wsp(size_t off) const { return reinterpret_cast<T *>(d_ws + off); }
};

namespace {

template <int D, int W, int S, bool kMulti>
int32_t launch_attention(ckv_pool *pool, const ckv::AttnParams &ap, cudaStream_t stream)
{
    using Lay = ckv::AttnLayout<D, W, S>;
    static thread_local int configured_device = -1;
    auto kernel = ckv::paged_decode_attn_kernel<D, W, S, kMulti>;
    if (configured_device != pool->device) {
        CKV_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay::kSmemBytes));
        configured_device = pool->device;
    }
    const int ctas = (pool->num_spans + W - 1) / W;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(ctas);
    lc.blockDim = dim3(Lay::kThreads);
    lc.dynamicSmemBytes = Lay::kSmemBytes;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pool->overlap ? 1 : 0;
    lc.attrs = attr;
    lc.numAttrs = 1;
    CKV_CUDA(cudaLaunchKernelEx(&lc, kernel, pool->tmap, ap));
    return CKV_OK;
}

int32_t check_device(const ckv_pool *pool, const char *fn)
{
    if (!pool) return fail(CKV_EINVAL, "%s: pool is NULL", fn);
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != pool->device)
        return fail(CKV_EINVAL, "%s: the pool lives on device %d but device %d is current", fn, pool->device, current);
    return CKV_OK;
}

int32_t check_call(ckv_pool *pool, int32_t layer, int32_t batch, const char *fn)
{
    if (int32_t rc = check_device(pool, fn)) return rc;
    if (layer < 0 || layer >= pool->cfg.num_layers)
        return fail(CKV_EINVAL, "%s: layer %d outside [0, %d)", fn, layer, pool->cfg.num_layers);
    if (batch < 1 || batch > pool->cfg.max_batch)
        return fail(CKV_EINVAL, "%s: batch %d outside [1, %d]", fn, batch, pool->cfg.max_batch);
    return CKV_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int32_t launch_plan(ckv_pool *pool, int32_t batch, const int32_t *d_seq_lens, cudaStream_t stream)
{
    const ckv_config &c = pool->cfg;
    ckv::PlanParams pp{};
    pp.seq_lens = d_seq_lens;
    pp.header = pool->wsp<ckv::PlanHeader>(pool->ws.header);
    pp.span_start = pool->wsp<int4>(pool->ws.span_start);
    pp.batch = batch;
    pp.max_pages_per_req = c.max_pages_per_req;
    pp.num_kv_heads = c.num_kv_heads;
    pp.num_spans = pool->num_spans;
    ckv::splitkv_plan_kernel<<<(pool->num_spans + 7) / 8, 256, 0, stream>>>(pp);
    CKV_CUDA(cudaGetLastError());
    pool->launches += 1;
    return CKV_OK;
}

// ------------------------------------------------------------------------------------------
// Scratch for decode_attention_noalloc: lives in the library image, one copy per GPU that loads
// it, for the life of the process.  Sized for kNoAllocMaxSpans spans at head_dim 128.
// ------------------------------------------------------------------------------------------
constexpr int kNoAllocMaxSpans = 640;
constexpr size_t kNaStatus = 0;                                                       // 256 B
constexpr size_t kNaArrivals = 256;                                                   // int32 [640]
constexpr size_t kNaSpanStart = kNaArrivals + sizeof(int32_t) * kNoAllocMaxSpans;     // int4 [640]
constexpr size_t kNaTrace = kNaSpanStart + sizeof(int4) * kNoAllocMaxSpans;           // u64 [640][8]
constexpr size_t kNaPart = kNaTrace + sizeof(unsigned long long) * 8 * kNoAllocMaxSpans;   // partial slots
constexpr size_t kNoAllocScratchBytes = kNaPart + sizeof(float) * 2 * kNoAllocMaxSpans * (2 * ckv::kMaxGroup + ckv::kMaxGroup * 128);
static_assert(kNaSpanStart % 16 == 0 && kNaTrace % 8 == 0 && kNaPart % 256 == 0,
              "sub-buffers of the static scratch must keep their natural alignment");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
// Device address of g_noalloc_scratch on each device (0 = not looked up yet).  In host code the
// symbol's name is only a handle; the address a kernel can use comes from cudaGetSymbolAddress.
unsigned char *g_noalloc_ptr[kMaxDevices] = {};

template <int D, int W, int NS>
int32_t launch_attention_noalloc(const CUtensorMap &tmap, const ckv::AttnParams &ap, cudaStream_t stream)
{
    using Lay = ckv::AttnLayout<D, W, NS>;
    auto kernel = ckv::paged_decode_attn_kernel<D, W, NS, false>;
    static bool configured[kMaxDevices] = {};                     // per device: the attribute is set once
    int device = 0;
    CKV_CUDA(cudaGetDevice(&device));
    if (!configured[device]) {
        CKV_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay::kSmemBytes));
        configured[device] = true;
    }
    kernel<<<(ap.num_spans + W - 1) / W, Lay::kThreads, Lay::kSmemBytes, stream>>>(tmap, ap);
    CKV_CUDA(cudaGetLastError());
    return CKV_OK;
}

template <int D, int W, int NS>
int32_t launch_read_probe(ckv_pool *pool, const ckv::ProbeParams &pp, cudaStream_t stream)
{
    using Lay = ckv::AttnLayout<D, W, NS>;
    auto kernel = ckv::pool_read_probe_kernel<D, W, NS>;
    static thread_local int configured_device = -1;
    if (configured_device != pool->device) {
        CKV_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay::kSmemBytes));
        configured_device = pool->device;
    }
    kernel<<<(pool->num_spans + W - 1) / W, W * 32, Lay::kSmemBytes, stream>>>(pool->tmap, pp);
    CKV_CUDA(cudaGetLastError());
    return CKV_OK;
}

}  // namespace

extern "C" {

const char *ckv_last_error(void) { return g_error; }

size_t kv_pool_bytes(const ckv_config *cfg)
{
    const char *why;
    if (!config_ok(cfg, &why)) { fail(CKV_EINVAL, "kv_pool_bytes: %s", why); return 0; }
    return (size_t)cfg->num_layers * cfg->num_pages * cfg->num_kv_heads * 2 * cfg->page_size * cfg->head_dim * 2;
}

size_t kv_workspace_bytes(const ckv_config *cfg)
{
    const char *why;
    if (!config_ok(cfg, &why)) { fail(CKV_EINVAL, "kv_workspace_bytes: %s", why); return 0; }
    return carve(*cfg).total;
}

int32_t kv_pool_create(const ckv_config *cfg, void *d_pool, size_t pool_bytes, void *d_workspace,
                       size_t workspace_bytes, int32_t device, ckv_pool **out_pool)
{
    const char *why;
    if (!out_pool) return fail(CKV_EINVAL, "kv_pool_create: out_pool is NULL");
    *out_pool = nullptr;
    if (!config_ok(cfg, &why)) return fail(CKV_EINVAL, "kv_pool_create: %s", why);
    if (!d_pool || !d_workspace) return fail(CKV_EINVAL, "kv_pool_create: NULL device buffer");
    if (reinterpret_cast<uintptr_t>(d_pool) & 255u) return fail(CKV_EINVAL, "kv_pool_create: d_pool not 256-byte aligned");
    if (reinterpret_cast<uintptr_t>(d_workspace) & 255u) return fail(CKV_EINVAL, "kv_pool_create: d_workspace not 256-byte aligned");
    if (pool_bytes < kv_pool_bytes(cfg)) return fail(CKV_ENOMEM, "kv_pool_create: pool buffer holds %zu bytes, %zu needed", pool_bytes, kv_pool_bytes(cfg));
    const WorkspaceLayout ws = carve(*cfg);
    if (workspace_bytes < ws.total) return fail(CKV_ENOMEM, "kv_pool_create: workspace holds %zu bytes, %zu needed", workspace_bytes, ws.total);
    if (device < 0) return fail(CKV_EINVAL, "kv_pool_create: device < 0");

    CKV_CUDA(cudaSetDevice(device));
    int cc_major = 0, sms = 0;
    CKV_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, device));
    CKV_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    if (cc_major != 10) return fail(CKV_ECUDA, "kv_pool_create: device %d is sm_%dx; this library is built for sm_100a only", device, cc_major);

    ckv_pool *p = new (std::nothrow) ckv_pool();
    if (!p) return fail(CKV_ENOMEM, "kv_pool_create: host allocation failed");
    p->cfg = *cfg;
    p->device = device;
    p->num_sms = sms;
    p->num_spans = std::min(sms * (cfg->head_dim == 128 ? kWarps128 : kWarps64), ckv::kMaxSpans);
    p->d_pool = static_cast<uint8_t *>(d_pool);
    p->d_ws = static_cast<uint8_t *>(d_workspace);
    p->ws = ws;
    p->launches = 0;
    p->profile = false;
    p->overlap = true;
    p->pool_written = false;
    p->inputs_from_predecessor = false;
    p->host_route = CKV_HOST_ROUTE_AUTO;
    p->ev_used = 0;

    if (int32_t rc = encode_pool_map(cfg, d_pool, &p->tmap, "kv_pool_create")) {
        delete p;
        return rc;
    }
    cudaError_t me = cudaMemset(d_workspace, 0, ws.total);
    if (me == cudaSuccess) me = cudaDeviceSynchronize();
    if (me != cudaSuccess) {
        delete p;
        return fail(CKV_ECUDA, "kv_pool_create: clearing the workspace failed: %s", cudaGetErrorString(me));
    }
    *out_pool = p;
    return CKV_OK;
}

int32_t kv_pool_destroy(ckv_pool *pool)
{
    if (!pool) return fail(CKV_EINVAL, "kv_pool_destroy: pool is NULL");
    cudaSetDevice(pool->device);
    cudaDeviceSynchronize();
    for (cudaEvent_t ev : pool->ev) cudaEventDestroy(ev);
    delete pool;
    return CKV_OK;
}

int32_t ckv_set_partition(ckv_pool *pool, int32_t num_spans)
{
    if (!pool) return fail(CKV_EINVAL, "ckv_set_partition: pool is NULL");
    if (num_spans < 1 || num_spans > ckv::kMaxSpans) return fail(CKV_EINVAL, "ckv_set_partition: %d outside [1, %d]", num_spans, ckv::kMaxSpans);
    pool->num_spans = num_spans;
    return CKV_OK;
}

int32_t ckv_get_partition(const ckv_pool *pool) { return pool ? pool->num_spans : CKV_EINVAL; }

int32_t ckv_set_overlap(ckv_pool *pool, int32_t enable)
{
    if (!pool) return fail(CKV_EINVAL, "ckv_set_overlap: pool is NULL");
    pool->overlap = enable != 0;
    return CKV_OK;
}

int32_t ckv_set_host_route(ckv_pool *pool, int32_t route)
{
    if (!pool) return fail(CKV_EINVAL, "ckv_set_host_route: pool is NULL");
    if (route < CKV_HOST_ROUTE_AUTO || route > CKV_HOST_ROUTE_COPY) return fail(CKV_EINVAL, "ckv_set_host_route: unknown route %d", route);
    pool->host_route = route;
    return CKV_OK;
}

int64_t ckv_launch_count(const ckv_pool *pool) { return pool ? pool->launches : 0; }

static int32_t append_launch(ckv_pool *pool, const char *fn, int32_t layer, int32_t batch, int32_t q_len,
                             const int32_t *d_block_tables, const int32_t *d_seq_lens, const void *d_k_new,
                             const void *d_v_new, void *stream)
{
    if (int32_t rc = check_call(pool, layer, batch, fn)) return rc;
    if (q_len < 1 || q_len > ckv::kMaxGroup) return fail(CKV_EINVAL, "%s: q_len %d outside [1, 8]", fn, q_len);
    if (!d_block_tables || !d_seq_lens || !d_k_new || !d_v_new) return fail(CKV_EINVAL, "%s: NULL argument", fn);
    if (!aligned16(d_k_new) || !aligned16(d_v_new)) return fail(CKV_EINVAL, "%s: k_new/v_new not 16-byte aligned", fn);
    const ckv_config &c = pool->cfg;
    ckv::AppendParams ap{};
    const size_t layer_bytes = (size_t)c.num_pages * c.num_kv_heads * 2 * c.page_size * c.head_dim * 2;
    ap.pool_layer = reinterpret_cast<uint4 *>(pool->d_pool + layer_bytes * layer);
    ap.block_tables = d_block_tables;
    ap.seq_lens = d_seq_lens;
    ap.k_new = static_cast<const uint4 *>(d_k_new);
    ap.v_new = static_cast<const uint4 *>(d_v_new);
    ap.status = pool->wsp<uint32_t>(pool->ws.status);
    ap.batch = batch;
    ap.max_pages_per_req = c.max_pages_per_req;
    ap.num_pages = c.num_pages;
    ap.num_kv_heads = c.num_kv_heads;
    ap.head_dim = c.head_dim;
    ap.q_len = q_len;
    const long long work = (long long)batch * q_len * c.num_kv_heads * 2 * (c.head_dim / 8);
    const int threads = 256;
    const int blocks = (int)std::min<long long>((work + threads - 1) / threads, 4096);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(blocks);
    lc.blockDim = dim3(threads);
    lc.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pool->overlap ? 1 : 0;
    lc.attrs = attr;
    lc.numAttrs = 1;
    CKV_CUDA(cudaLaunchKernelEx(&lc, ckv::kv_append_kernel, ap));
    pool->launches += 1;
    pool->pool_written = true;
    return CKV_OK;
}

int32_t kv_append(ckv_pool *pool, int32_t layer, int32_t batch, const int32_t *d_block_tables,
                  const int32_t *d_seq_lens, const void *d_k_new, const void *d_v_new, void *stream)
{
    return append_launch(pool, "kv_append", layer, batch, 1, d_block_tables, d_seq_lens, d_k_new, d_v_new, stream);
}

int32_t kv_append_multi(ckv_pool *pool, int32_t layer, int32_t batch, int32_t q_len, const int32_t *d_block_tables,
                        const int32_t *d_seq_lens, const void *d_k_new, const void *d_v_new, void *stream)
{
    return append_launch(pool, "kv_append_multi", layer, batch, q_len, d_block_tables, d_seq_lens, d_k_new, d_v_new,
                         stream);
}

// Attention for one layer, optionally with the KV append folded into the same kernel.
static int32_t attention_launch(ckv_pool *pool, const char *fn, int32_t layer, int32_t batch, int32_t q_len,
                                const int32_t *d_block_tables, const int32_t *d_seq_lens, const void *d_q,
                                const void *d_k_new, const void *d_v_new, void *d_out, void *stream)
{
    if (int32_t rc = check_call(pool, layer, batch, fn)) return rc;
    if (q_len < 1 || q_len > ckv::kMaxGroup) return fail(CKV_EINVAL, "%s: q_len %d outside [1, %d]", fn, q_len, ckv::kMaxGroup);
    if (q_len > 1 && d_k_new) return fail(CKV_EINVAL, "%s: the fused append is for single-token steps", fn);
    if (!d_block_tables || !d_seq_lens || !d_q || !d_out) return fail(CKV_EINVAL, "%s: NULL argument", fn);
    if (!aligned16(d_q) || !aligned16(d_out)) return fail(CKV_EINVAL, "%s: q/out not 16-byte aligned", fn);
    if ((d_k_new == nullptr) != (d_v_new == nullptr)) return fail(CKV_EINVAL, "%s: k_new and v_new go together", fn);
    if (d_k_new && (!aligned16(d_k_new) || !aligned16(d_v_new))) return fail(CKV_EINVAL, "%s: k_new/v_new not 16-byte aligned", fn);
    const ckv_config &c = pool->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    ckv::AttnParams ap{};
    ap.block_tables = d_block_tables;
    ap.seq_lens = d_seq_lens;
    ap.q = static_cast<const uint16_t *>(d_q);
    ap.out = static_cast<uint16_t *>(d_out);
    ap.k_new = static_cast<const uint4 *>(d_k_new);
    ap.v_new = static_cast<const uint4 *>(d_v_new);
    ap.pool_layer = d_k_new ? reinterpret_cast<uint4 *>(pool->d_pool + (size_t)c.num_pages * c.num_kv_heads * 2 * c.page_size * c.head_dim * 2 * layer)
                            : nullptr;
    ap.part = pool->wsp<float>(pool->ws.part);
    ap.arrivals = pool->wsp<int32_t>(pool->ws.arrivals);
    ap.span_start = pool->wsp<int4>(pool->ws.span_start);
    ap.trace = pool->wsp<unsigned long long>(pool->ws.trace);
    ap.status = pool->wsp<uint32_t>(pool->ws.status);
    ap.batch = batch;
    ap.max_pages_per_req = c.max_pages_per_req;
    ap.num_pages = c.num_pages;
    ap.num_kv_heads = c.num_kv_heads;
    ap.num_q_heads = c.num_q_heads;
    ap.group = c.num_q_heads / c.num_kv_heads;
    ap.layer_page_base = layer * c.num_pages;
    ap.num_spans = pool->num_spans;
    ap.q_len = q_len;
    ap.q_base = 0;
    ap.q_pass = q_len;
    // A fused step may start loading tiles under its predecessor's tail -- unless that predecessor
    // may be a kernel of this library that writes the pool (an append or a swap-in).
    ap.early_loads = pool->inputs_from_predecessor ? -1 : pool->pool_written ? 0 : 1;
    pool->pool_written = false;
    pool->inputs_from_predecessor = false;
    ap.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)c.head_dim));

    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (pool->profile && pool->ev_used < kMaxProfile) {
        if ((size_t)(2 * pool->ev_used + 2) > pool->ev.size()) {
            cudaEvent_t a = nullptr, b = nullptr;
            CKV_CUDA(cudaEventCreate(&a));
            const cudaError_t ce = cudaEventCreate(&b);
            if (ce != cudaSuccess) {
                cudaEventDestroy(a);
                return fail(CKV_ECUDA, "%s: cudaEventCreate failed: %s", fn, cudaGetErrorString(ce));
            }
            pool->ev.push_back(a);
            pool->ev.push_back(b);
        }
        ev0 = pool->ev[2 * pool->ev_used];
        ev1 = pool->ev[2 * pool->ev_used + 1];
        pool->ev_used += 1;
        CKV_CUDA(cudaEventRecord(ev0, s));
    }
    // One launch holds 8 (new token, head) columns: 8 / group new tokens.  More new tokens take
    // more launches, each streaming the KV again for its own block of new tokens.
    const int per_pass = ckv::kMaxGroup / ap.group;
    for (int base = 0; base < q_len; base += per_pass) {
        ap.q_base = base;
        ap.q_pass = std::min(per_pass, q_len - base);
        int32_t rc;
        if (c.head_dim == 128)
            rc = q_len > 1 ? launch_attention<128, kWarps128, kStages128, true>(pool, ap, s)
                           : launch_attention<128, kWarps128, kStages128, false>(pool, ap, s);
        else
            rc = q_len > 1 ? launch_attention<64, kWarps64, kStages64, true>(pool, ap, s)
                           : launch_attention<64, kWarps64, kStages64, false>(pool, ap, s);
        if (rc) return rc;
        pool->launches += 1;
    }
    if (ev1) CKV_CUDA(cudaEventRecord(ev1, s));
    return CKV_OK;
}

int32_t decode_attention(ckv_pool *pool, int32_t layer, int32_t batch, const int32_t *d_block_tables,
                         const int32_t *d_seq_lens, const void *d_q, void *d_out, void *stream)
{
    return attention_launch(pool, "decode_attention", layer, batch, 1, d_block_tables, d_seq_lens, d_q, nullptr,
                            nullptr, d_out, stream);
}

int32_t decode_attention_multi(ckv_pool *pool, int32_t layer, int32_t batch, int32_t q_len,
                               const int32_t *d_block_tables, const int32_t *d_seq_lens, const void *d_q,
                               void *d_out, void *stream)
{
    return attention_launch(pool, "decode_attention_multi", layer, batch, q_len, d_block_tables, d_seq_lens, d_q,
                            nullptr, nullptr, d_out, stream);
}

int32_t decode_step(ckv_pool *pool, int32_t layer, int32_t batch, const int32_t *d_block_tables,
                    const int32_t *d_seq_lens, const void *d_q, const void *d_k_new, const void *d_v_new,
                    void *d_out, void *stream)
{
    if (!d_k_new || !d_v_new) return fail(CKV_EINVAL, "decode_step: NULL k_new/v_new");
    return attention_launch(pool, "decode_step", layer, batch, 1, d_block_tables, d_seq_lens, d_q, d_k_new, d_v_new,
                            d_out, stream);
}

int32_t kv_read_probe(ckv_pool *pool, int32_t layer, int32_t batch, const int32_t *d_block_tables,
                      const int32_t *d_seq_lens, void *stream)
{
    if (int32_t rc = check_call(pool, layer, batch, "kv_read_probe")) return rc;
    if (!d_block_tables || !d_seq_lens) return fail(CKV_EINVAL, "kv_read_probe: NULL argument");
    const ckv_config &c = pool->cfg;
    ckv::ProbeParams pp{};
    pp.block_tables = d_block_tables;
    pp.seq_lens = d_seq_lens;
    pp.status = pool->wsp<uint32_t>(pool->ws.status);
    pp.sink = reinterpret_cast<unsigned long long *>(pool->d_ws + pool->ws.status + 64);
    pp.batch = batch;
    pp.max_pages_per_req = c.max_pages_per_req;
    pp.num_pages = c.num_pages;
    pp.num_kv_heads = c.num_kv_heads;
    pp.layer_page_base = layer * c.num_pages;
    pp.num_spans = pool->num_spans;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int32_t rc = c.head_dim == 128 ? launch_read_probe<128, kWarps128, kStages128>(pool, pp, s)
                                         : launch_read_probe<64, kWarps64, kStages64>(pool, pp, s);
    if (rc) return rc;
    pool->launches += 1;
    return CKV_OK;
}

int32_t decode_plan(ckv_pool *pool, int32_t batch, const int32_t *d_seq_lens, void *stream,
                    int32_t *h_header, int32_t *h_span_start)
{
    if (int32_t rc = check_call(pool, 0, batch, "decode_plan")) return rc;
    if (!d_seq_lens || !h_header || !h_span_start) return fail(CKV_EINVAL, "decode_plan: NULL argument");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int32_t rc = launch_plan(pool, batch, d_seq_lens, s)) return rc;
    CKV_CUDA(cudaMemcpyAsync(h_header, pool->d_ws + pool->ws.header, sizeof(ckv::PlanHeader), cudaMemcpyDeviceToHost, s));
    CKV_CUDA(cudaMemcpyAsync(h_span_start, pool->d_ws + pool->ws.span_start, sizeof(int4) * pool->num_spans, cudaMemcpyDeviceToHost, s));
    CKV_CUDA(cudaStreamSynchronize(s));
    return CKV_OK;
}

int32_t kv_check_status(ckv_pool *pool, void *stream, uint32_t *out_bits)
{
    if (int32_t rc = check_device(pool, "kv_check_status")) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t bits = 0;
    CKV_CUDA(cudaMemcpyAsync(&bits, pool->d_ws + pool->ws.status, sizeof bits, cudaMemcpyDeviceToHost, s));
    CKV_CUDA(cudaMemsetAsync(pool->d_ws + pool->ws.status, 0, sizeof bits, s));
    CKV_CUDA(cudaStreamSynchronize(s));
    if (out_bits) *out_bits = bits;
    if (bits & ckv::kStatusWaitLimit) {
        // a warp that gave up may have left arrival counters half-way; start the next launch clean
        CKV_CUDA(cudaMemsetAsync(pool->d_ws + pool->ws.arrivals, 0, sizeof(int32_t) * ckv::kMaxSpans, s));
        CKV_CUDA(cudaStreamSynchronize(s));
    }
    if (bits & ckv::kStatusWaitLimit) return fail(CKV_ETIMEOUT, "device status 0x%x: a bounded wait gave up", bits);
    if (bits & (ckv::kStatusBadLength | ckv::kStatusBadPage))
        return fail(CKV_EBOUNDS, "device status 0x%x: %s%s", bits, (bits & ckv::kStatusBadLength) ? "[context length out of range]" : "",
                    (bits & ckv::kStatusBadPage) ? "[page id out of range]" : "");
    return CKV_OK;
}

int32_t ckv_wait_limit_selftest(ckv_pool *pool, uint64_t limit_ns, void *stream)
{
    if (int32_t rc = check_device(pool, "ckv_wait_limit_selftest")) return rc;
    if (limit_ns < 1000 || limit_ns > 100000000ull)
        return fail(CKV_EINVAL, "ckv_wait_limit_selftest: limit outside [1 us, 100 ms]");
    ckv::wait_limit_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        pool->wsp<uint32_t>(pool->ws.status), pool->wsp<int32_t>(pool->ws.arrivals), limit_ns);
    CKV_CUDA(cudaGetLastError());
    pool->launches += 1;
    return CKV_OK;
}

// Device-visible address of a host buffer if the device can address it (pinned or registered
// memory), else NULL.
static void *mapped_or_null(const void *h)
{
    void *d = nullptr;
    if (cudaHostGetDevicePointer(&d, const_cast<void *>(h), 0) != cudaSuccess) {
        cudaGetLastError();                      // not an error of the caller's: the copy path is taken
        return nullptr;
    }
    return d;
}

int32_t decode_step_host(ckv_pool *pool, int32_t layer, int32_t batch, const int32_t *h_block_tables,
                         const int32_t *h_seq_lens, const void *h_q, const void *h_k_new,
                         const void *h_v_new, void *h_out, void *stream)
{
    if (int32_t rc = check_call(pool, layer, batch, "decode_step_host")) return rc;
    if (!h_block_tables || !h_seq_lens || !h_q || !h_k_new || !h_v_new || !h_out)
        return fail(CKV_EINVAL, "decode_step_host: NULL argument");
    const ckv_config &c = pool->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t d2 = (size_t)c.head_dim * 2;
    int32_t *d_bt = pool->wsp<int32_t>(pool->ws.st_tables);
    int32_t *d_sl = pool->wsp<int32_t>(pool->ws.st_lens);
    void *d_q = pool->d_ws + pool->ws.st_q, *d_k = pool->d_ws + pool->ws.st_k;
    void *d_v = pool->d_ws + pool->ws.st_v, *d_o = pool->d_ws + pool->ws.st_out;
    const size_t n_bt = sizeof(int32_t) * (size_t)batch * c.max_pages_per_req, n_sl = sizeof(int32_t) * (size_t)batch;
    const size_t n_q = (size_t)batch * c.num_q_heads * d2, n_kv = (size_t)batch * c.num_kv_heads * d2;

    // Pinned buffers the device can address take one of two routes without a DMA copy; both write
    // the output rows straight into the host buffer.
    //   staged: one gather kernel brings the five inputs into the workspace, the attention kernel
    //           follows it with programmatic serialization and waits for it before its plan;
    //   direct: the attention kernel reads tables, lengths, q and the new rows straight from host
    //           memory (one launch; every read crosses the host link with its latency).
    const void *m_bt = mapped_or_null(h_block_tables), *m_sl = mapped_or_null(h_seq_lens), *m_q = mapped_or_null(h_q);
    const void *m_k = mapped_or_null(h_k_new), *m_v = mapped_or_null(h_v_new);
    void *m_o = mapped_or_null(h_out);
    const bool all_mapped = m_bt && m_sl && m_q && m_k && m_v && m_o && aligned16(m_o);
    const bool direct_ok = all_mapped && aligned16(m_q) && aligned16(m_k) && aligned16(m_v);
    if (direct_ok && pool->host_route == CKV_HOST_ROUTE_DIRECT) {
        const int32_t rc = decode_step(pool, layer, batch, static_cast<const int32_t *>(m_bt), static_cast<const int32_t *>(m_sl),
                                       m_q, m_k, m_v, m_o, stream);
        if (rc) return rc;
        CKV_CUDA(cudaStreamSynchronize(s));
        return CKV_OK;
    }
    if (all_mapped && pool->host_route != CKV_HOST_ROUTE_COPY) {
        ckv::GatherParams gp{};
        const void *src[5] = {m_bt, m_sl, m_q, m_k, m_v};
        void *dst[5] = {d_bt, d_sl, d_q, d_k, d_v};
        const size_t bytes[5] = {n_bt, n_sl, n_q, n_kv, n_kv};
        size_t total = 0;
        for (int a = 0; a < 5; ++a) {
            gp.src[a] = static_cast<const uint8_t *>(src[a]);
            gp.dst[a] = static_cast<uint8_t *>(dst[a]);
            gp.bytes[a] = bytes[a];
            total += bytes[a];
        }
        const int blocks = (int)std::min<size_t>((total / 16 + 255) / 256 + 1, (size_t)pool->num_sms * 8);
        ckv::host_gather_kernel<<<blocks, 256, 0, s>>>(gp);
        CKV_CUDA(cudaGetLastError());
        pool->launches += 1;
        pool->inputs_from_predecessor = true;    // the attention kernel starts under the gather and waits for it first
        const int32_t rc = decode_step(pool, layer, batch, d_bt, d_sl, d_q, d_k, d_v, m_o, stream);
        if (rc) return rc;
        CKV_CUDA(cudaStreamSynchronize(s));
        return CKV_OK;
    }

    CKV_CUDA(cudaMemcpyAsync(d_bt, h_block_tables, n_bt, cudaMemcpyHostToDevice, s));
    CKV_CUDA(cudaMemcpyAsync(d_sl, h_seq_lens, n_sl, cudaMemcpyHostToDevice, s));
    CKV_CUDA(cudaMemcpyAsync(d_q, h_q, n_q, cudaMemcpyHostToDevice, s));
    CKV_CUDA(cudaMemcpyAsync(d_k, h_k_new, n_kv, cudaMemcpyHostToDevice, s));
    CKV_CUDA(cudaMemcpyAsync(d_v, h_v_new, n_kv, cudaMemcpyHostToDevice, s));
    if (int32_t rc = decode_step(pool, layer, batch, d_bt, d_sl, d_q, d_k, d_v, d_o, stream)) return rc;
    CKV_CUDA(cudaMemcpyAsync(h_out, d_o, n_q, cudaMemcpyDeviceToHost, s));
    CKV_CUDA(cudaStreamSynchronize(s));
    return CKV_OK;
}

int32_t step_latency_sweep(ckv_pool *pool, int32_t n_sizes, const int32_t *batch_sizes, int32_t batch_stride,
                           const int32_t *d_block_tables, const int32_t *d_seq_lens, const void *d_q,
                           const void *d_k_new, const void *d_v_new, void *d_out, int32_t warmup,
                           int32_t iters, void *d_flush, size_t flush_bytes, void *stream,
                           double *out_median_us, double *out_min_us)
{
    if (int32_t rc = check_device(pool, "step_latency_sweep")) return rc;
    if (n_sizes < 1 || !batch_sizes || !out_median_us || !out_min_us) return fail(CKV_EINVAL, "step_latency_sweep: bad size list or outputs");
    if (warmup < 0 || iters < 1 || iters > 100000) return fail(CKV_EINVAL, "step_latency_sweep: bad warmup/iters");
    if (batch_stride < 1 || batch_stride > pool->cfg.max_batch) return fail(CKV_EINVAL, "step_latency_sweep: bad batch_stride");
    for (int i = 0; i < n_sizes; ++i)
        if (batch_sizes[i] < 1 || batch_sizes[i] > batch_stride) return fail(CKV_EINVAL, "step_latency_sweep: batch size %d outside [1, %d]", batch_sizes[i], batch_stride);
    if (!d_block_tables || !d_seq_lens || !d_q || !d_k_new || !d_v_new || !d_out) return fail(CKV_EINVAL, "step_latency_sweep: NULL argument");
    const ckv_config &c = pool->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t d2 = (size_t)c.head_dim * 2;
    const size_t q_layer = (size_t)batch_stride * c.num_q_heads * d2;
    const size_t kv_layer = (size_t)batch_stride * c.num_kv_heads * d2;

    std::vector<cudaEvent_t> ev(2 * (size_t)iters, nullptr);
    int32_t rc = CKV_OK;
    for (auto &e : ev) {
        const cudaError_t ce = cudaEventCreate(&e);
        if (ce != cudaSuccess) {
            e = nullptr;
            rc = fail(CKV_ECUDA, "step_latency_sweep: cudaEventCreate failed: %s", cudaGetErrorString(ce));
            break;
        }
    }
    auto record = [&](cudaEvent_t e) {
        const cudaError_t ce = cudaEventRecord(e, s);
        if (ce != cudaSuccess && rc == CKV_OK) rc = fail(CKV_ECUDA, "step_latency_sweep: cudaEventRecord failed: %s", cudaGetErrorString(ce));
    };
    std::vector<float> ms((size_t)iters);
    for (int i = 0; i < n_sizes && rc == CKV_OK; ++i) {
        const int32_t b = batch_sizes[i];
        for (int k = 0; k < warmup + iters && rc == CKV_OK; ++k) {
            const bool timed = k >= warmup;
            if (d_flush && flush_bytes) {
                // overwrite the first half (evicts everything), then read the second half (leaves the
                // cache holding clean lines instead of the overwrite's dirty ones)
                const size_t half = (flush_bytes / 2) & ~(size_t)15;
                cudaError_t e = cudaMemsetAsync(d_flush, k & 0xff, half, s);
                if (e != cudaSuccess) { rc = fail(CKV_ECUDA, "flush memset failed: %s", cudaGetErrorString(e)); break; }
                ckv::l2_read_sweep_kernel<<<4 * pool->num_sms, 256, 0, s>>>(
                    reinterpret_cast<const uint4 *>(static_cast<const uint8_t *>(d_flush) + half), half / 16,
                    static_cast<uint32_t *>(d_flush));
                e = cudaGetLastError();
                if (e != cudaSuccess) { rc = fail(CKV_ECUDA, "flush read sweep failed: %s", cudaGetErrorString(e)); break; }
            }
            if (timed) record(ev[2 * (size_t)(k - warmup)]);
            for (int layer = 0; layer < c.num_layers && rc == CKV_OK; ++layer) {
                const uint8_t *q = static_cast<const uint8_t *>(d_q) + q_layer * layer;
                const uint8_t *kn = static_cast<const uint8_t *>(d_k_new) + kv_layer * layer;
                const uint8_t *vn = static_cast<const uint8_t *>(d_v_new) + kv_layer * layer;
                uint8_t *o = static_cast<uint8_t *>(d_out) + q_layer * layer;
                rc = decode_step(pool, layer, b, d_block_tables, d_seq_lens, q, kn, vn, o, stream);
            }
            if (timed) record(ev[2 * (size_t)(k - warmup) + 1]);
        }
        if (rc != CKV_OK) break;
        cudaError_t e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) { rc = fail(CKV_ECUDA, "step_latency_sweep: synchronise failed: %s", cudaGetErrorString(e)); break; }
        for (int k = 0; k < iters && rc == CKV_OK; ++k) {
            const cudaError_t ce = cudaEventElapsedTime(&ms[k], ev[2 * (size_t)k], ev[2 * (size_t)k + 1]);
            if (ce != cudaSuccess) rc = fail(CKV_ECUDA, "step_latency_sweep: cudaEventElapsedTime failed: %s", cudaGetErrorString(ce));
        }
        if (rc != CKV_OK) break;
        std::vector<float> sorted(ms);
        std::sort(sorted.begin(), sorted.end());
        const double med = (iters & 1) ? sorted[iters / 2] : 0.5 * (sorted[iters / 2 - 1] + sorted[iters / 2]);
        out_median_us[i] = med * 1000.0;
        out_min_us[i] = sorted[0] * 1000.0;
    }
    for (auto &e : ev)
        if (e) cudaEventDestroy(e);
    if (rc != CKV_OK) return rc;
    return kv_check_status(pool, stream, nullptr);
}

int32_t ckv_read_span_trace(ckv_pool *pool, void *stream, uint64_t *h_trace, int32_t *h_span_start)
{
    if (!pool || !h_trace) return fail(CKV_EINVAL, "ckv_read_span_trace: NULL argument");
    if (int32_t rc = check_device(pool, "ckv_read_span_trace")) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CKV_CUDA(cudaMemcpyAsync(h_trace, pool->d_ws + pool->ws.trace, sizeof(uint64_t) * 8 * pool->num_spans,
                             cudaMemcpyDeviceToHost, s));
    if (h_span_start)
        CKV_CUDA(cudaMemcpyAsync(h_span_start, pool->d_ws + pool->ws.span_start, sizeof(int4) * pool->num_spans,
                                 cudaMemcpyDeviceToHost, s));
    CKV_CUDA(cudaStreamSynchronize(s));
    return CKV_OK;
}

int32_t ckv_profile_enable(ckv_pool *pool, int32_t enable)
{
    if (!pool) return fail(CKV_EINVAL, "ckv_profile_enable: pool is NULL");
    pool->profile = enable != 0;
    pool->ev_used = 0;
    return CKV_OK;
}

int32_t ckv_profile_read(ckv_pool *pool, double *out_attention_ms, int32_t *out_launches)
{
    if (!pool || !out_attention_ms || !out_launches) return fail(CKV_EINVAL, "ckv_profile_read: NULL argument");
    CKV_CUDA(cudaSetDevice(pool->device));
    CKV_CUDA(cudaDeviceSynchronize());
    double total = 0.0;
    for (int i = 0; i < pool->ev_used; ++i) {
        float ms = 0.f;
        CKV_CUDA(cudaEventElapsedTime(&ms, pool->ev[2 * i], pool->ev[2 * i + 1]));
        total += ms;
    }
    *out_attention_ms = total;
    *out_launches = pool->ev_used;
    return CKV_OK;
}

int32_t decode_attention_noalloc(const ckv_config *cfg, const void *d_pool, int32_t layer, int32_t batch,
                                 const int32_t *d_block_tables, const int32_t *d_seq_lens, const void *d_q,
                                 void *d_out, int32_t num_spans, void *stream, uint32_t *h_status)
{
    const char *why;
    if (!config_ok(cfg, &why)) return fail(CKV_EINVAL, "decode_attention_noalloc: %s", why);
    if (!d_pool || !d_block_tables || !d_seq_lens || !d_q || !d_out)
        return fail(CKV_EINVAL, "decode_attention_noalloc: NULL argument");
    if (reinterpret_cast<uintptr_t>(d_pool) & 255u) return fail(CKV_EINVAL, "decode_attention_noalloc: d_pool not 256-byte aligned");
    if (!aligned16(d_q) || !aligned16(d_out)) return fail(CKV_EINVAL, "decode_attention_noalloc: q/out not 16-byte aligned");
    if (layer < 0 || layer >= cfg->num_layers) return fail(CKV_EINVAL, "decode_attention_noalloc: layer %d outside [0, %d)", layer, cfg->num_layers);
    if (batch < 1 || batch > cfg->max_batch) return fail(CKV_EINVAL, "decode_attention_noalloc: batch %d outside [1, %d]", batch, cfg->max_batch);

    int device = -1;
    CKV_CUDA(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return fail(CKV_EINVAL, "decode_attention_noalloc: device ordinal %d not supported", device);
    static int cached_cc[kMaxDevices] = {}, cached_sms[kMaxDevices] = {};      // looked up on a device's first call
    if (cached_sms[device] == 0) {
        int cc = 0, n = 0;
        CKV_CUDA(cudaDeviceGetAttribute(&cc, cudaDevAttrComputeCapabilityMajor, device));
        CKV_CUDA(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device));
        cached_cc[device] = cc;
        cached_sms[device] = n;
    }
    const int cc_major = cached_cc[device], sms = cached_sms[device];
    if (cc_major != 10) return fail(CKV_ECUDA, "decode_attention_noalloc: device %d is sm_%dx; this library is built for sm_100a only", device, cc_major);

    const int warps = cfg->head_dim == 128 ? kWarps128 : kWarps64;
    if (num_spans == 0) num_spans = sms * warps;
    if (num_spans < 1 || num_spans > kNoAllocMaxSpans)
        return fail(CKV_EINVAL, "decode_attention_noalloc: %d spans requested, the built-in scratch holds partial results "
                                "for at most %d (use decode_attention with a caller-provided workspace for more)",
                    num_spans, kNoAllocMaxSpans);

    // One-time set-up per device: the device address of the static scratch.
    if (g_noalloc_ptr[device] == nullptr) {
        unsigned char *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr)
            return fail(CKV_ECUDA, "decode_attention_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        g_noalloc_ptr[device] = ptr;
    }
    unsigned char *scratch = g_noalloc_ptr[device];

    // Tensor map over the caller's pool, built on the stack (a host-side encode, no allocation).
    CUtensorMap tmap;
    if (int32_t rc = encode_pool_map(cfg, d_pool, &tmap, "decode_attention_noalloc")) return rc;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The scratch keeps whatever the previous call left: the status word and the arrival counters
    // must start at zero (partials, span starts and the timeline are fully rewritten before use).
    CKV_CUDA(cudaMemsetAsync(scratch + kNaStatus, 0, kNaSpanStart - kNaStatus, s));

    ckv::AttnParams ap{};
    ap.block_tables = d_block_tables;
    ap.seq_lens = d_seq_lens;
    ap.q = static_cast<const uint16_t *>(d_q);
    ap.out = static_cast<uint16_t *>(d_out);
    ap.part = reinterpret_cast<float *>(scratch + kNaPart);
    ap.arrivals = reinterpret_cast<int32_t *>(scratch + kNaArrivals);
    ap.span_start = reinterpret_cast<int4 *>(scratch + kNaSpanStart);
    ap.trace = reinterpret_cast<unsigned long long *>(scratch + kNaTrace);
    ap.status = reinterpret_cast<uint32_t *>(scratch + kNaStatus);
    ap.batch = batch;
    ap.max_pages_per_req = cfg->max_pages_per_req;
    ap.num_pages = cfg->num_pages;
    ap.num_kv_heads = cfg->num_kv_heads;
    ap.num_q_heads = cfg->num_q_heads;
    ap.group = cfg->num_q_heads / cfg->num_kv_heads;
    ap.layer_page_base = layer * cfg->num_pages;
    ap.num_spans = num_spans;
    ap.q_len = 1;
    ap.q_base = 0;
    ap.q_pass = 1;
    ap.early_loads = 0;
    ap.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)cfg->head_dim));

    int32_t rc;
    if (cfg->head_dim == 128) rc = launch_attention_noalloc<128, kWarps128, kStages128>(tmap, ap, s);
    else rc = launch_attention_noalloc<64, kWarps64, kStages64>(tmap, ap, s);
    if (rc) return rc;

    if (h_status) {
        CKV_CUDA(cudaMemcpyAsync(h_status, scratch + kNaStatus, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
        CKV_CUDA(cudaStreamSynchronize(s));
        if (*h_status & ckv::kStatusWaitLimit) return fail(CKV_ETIMEOUT, "device status 0x%x: a bounded wait gave up", *h_status);
        if (*h_status) return fail(CKV_EBOUNDS, "device status 0x%x: context length or page id out of range", *h_status);
    }
    return CKV_OK;
}

static int32_t swap_launch(ckv_pool *pool, const char *fn, bool to_host, int32_t n_pages, const int32_t *d_page_ids,
                           void *h_image, size_t image_bytes, void *stream)
{
    if (int32_t rc = check_device(pool, fn)) return rc;
    if (n_pages < 1 || !d_page_ids || !h_image) return fail(CKV_EINVAL, "%s: bad page list or image", fn);
    const ckv_config &c = pool->cfg;
    const size_t page_bytes = (size_t)c.num_kv_heads * 2 * c.page_size * c.head_dim * 2;
    const size_t need = (size_t)c.num_layers * n_pages * page_bytes;
    if (image_bytes < need) return fail(CKV_ENOMEM, "%s: image holds %zu bytes, %zu needed", fn, image_bytes, need);
    if (reinterpret_cast<uintptr_t>(h_image) & 15u) return fail(CKV_EINVAL, "%s: image not 16-byte aligned", fn);
    void *d_image = nullptr;
    cudaError_t e = cudaHostGetDevicePointer(&d_image, h_image, 0);
    if (e != cudaSuccess || !d_image) {
        cudaGetLastError();
        return fail(CKV_EINVAL, "%s: the image must be pinned host memory the device can address (%s)", fn,
                    cudaGetErrorString(e));
    }
    ckv::SwapParams sp{};
    sp.pool = reinterpret_cast<uint4 *>(pool->d_pool);
    sp.image = static_cast<uint4 *>(d_image);
    sp.page_ids = d_page_ids;
    sp.status = pool->wsp<uint32_t>(pool->ws.status);
    sp.n_pages = n_pages;
    sp.num_layers = c.num_layers;
    sp.num_pages = c.num_pages;
    sp.page_vecs = (int32_t)(page_bytes / 16);
    const long long work = (long long)need / 16;
    const int threads = 256;
    const int blocks = (int)std::min<long long>((work + threads - 1) / threads, (long long)pool->num_sms * 8);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (to_host) ckv::kv_swap_kernel<true><<<blocks, threads, 0, s>>>(sp);
    else ckv::kv_swap_kernel<false><<<blocks, threads, 0, s>>>(sp);
    if (!to_host) pool->pool_written = true;
    CKV_CUDA(cudaGetLastError());
    pool->launches += 1;
    return CKV_OK;
}

int32_t kv_swap_out(ckv_pool *pool, int32_t n_pages, const int32_t *d_page_ids, void *h_image, size_t image_bytes,
                    void *stream)
{
    return swap_launch(pool, "kv_swap_out", true, n_pages, d_page_ids, h_image, image_bytes, stream);
}

int32_t kv_swap_in(ckv_pool *pool, int32_t n_pages, const int32_t *d_page_ids, const void *h_image,
                   size_t image_bytes, void *stream)
{
    return swap_launch(pool, "kv_swap_in", false, n_pages, d_page_ids, const_cast<void *>(h_image), image_bytes, stream);
}

}  // extern "C"
