/*
 * fp64 CPU oracle for one decode iteration's attention over a paged bf16 KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the GPU library
 * must compute.  It shares no code, header, table or helper with the CUDA path and is never
 * linked into, imported by or called from it.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may build or call it.
 *
 * What it states (paper, Section 2.1 "Inference Primer": each generated token depends on the
 * key and value vectors of all previous tokens of its sequence, which are kept in the KV cache;
 * Section 2.1 "PagedAttention": the cache is held in dynamically allocated pages), with the
 * arithmetic the hot path is defined by -- for request r, query head h, KV head kh = h / G:
 *
 *     s_j   = (1/sqrt(d)) * sum_c q[r][h][c] * k_j[c]            j = 0 .. L_r-1
 *     w_j   = exp(s_j - max_j s_j),   Z = sum_j w_j
 *     out[r][h][c] = ( sum_j w_j * v_j[c] ) / Z
 *
 * where k_j, v_j are token j's rows, found through the request's block table:
 * page = block_table[r][j / P], slot = j % P.
 *
 * Every function below is pinned by tests that do not re-use its own formula: hand-computed
 * cases, closed forms (L = 1, q = 0, one dominant key), softmax shift invariance, page
 * permutation invariance, split+combine equality, a dense brute force written separately in
 * numpy and torch's float64 softmax.  No function here is "parity unpinned".
 *
 * KV pool byte format (a data format both sides read, each through its own indexing code):
 *     bf16 pool[num_layers][num_pages][num_kv_heads][2 (0 = K, 1 = V)][page_size][head_dim]
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE-754 binary32: widening to double is exact. */
static double bf16_bits_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Number of threads the parallel loops below will use. */
int32_t oracle_num_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * The definition itself, on dense (already gathered) fp64 rows.
 *   q[d], K[L][d], V[L][d]  ->  out[d];  weights (optional, may be NULL) receives w_j / Z.
 * Two passes: all scores, their maximum, then the weights and the weighted mean.
 * Returns 0, or -1 on L < 1 / d < 1.
 */
int32_t oracle_attention_dense_f64(const double *q, const double *K, const double *V,
                                   int64_t L, int32_t d, double scale,
                                   double *out, double *weights)
{
    if (L < 1 || d < 1) return -1;
    double *s = (double *)malloc((size_t)L * sizeof(double));
    if (!s) return -2;

    double m = -INFINITY;
    for (int64_t j = 0; j < L; ++j) {
        double dot = 0.0;
        for (int32_t c = 0; c < d; ++c) dot += q[c] * K[j * d + c];
        s[j] = scale * dot;
        if (s[j] > m) m = s[j];
    }

    double Z = 0.0;
    for (int64_t j = 0; j < L; ++j) {
        s[j] = exp(s[j] - m);           /* s now holds w_j */
        Z += s[j];
    }

    for (int32_t c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int64_t j = 0; j < L; ++j) acc += s[j] * V[j * d + c];
        out[c] = acc / Z;
    }
    if (weights)
        for (int64_t j = 0; j < L; ++j) weights[j] = s[j] / Z;

    free(s);
    return 0;
}

/*
 * The same result reached through split-KV partials and a log-sum-exp combine: the context
 * [0, L) is cut at cuts[0] < cuts[1] < ... (each in (0, L)), every chunk i yields
 *     m_i = max s_j,  l_i = sum exp(s_j - m_i),  acc_i[c] = sum exp(s_j - m_i) v_j[c]
 * and the chunks are merged by
 *     m* = max_i m_i,  Z = sum_i l_i e^{m_i - m*},  out[c] = sum_i acc_i[c] e^{m_i - m*} / Z.
 * Mathematically equal to oracle_attention_dense_f64 for every choice of cuts.
 * Returns 0, or -1 on bad arguments.
 */
int32_t oracle_attention_split_f64(const double *q, const double *K, const double *V,
                                   int64_t L, int32_t d, double scale,
                                   const int64_t *cuts, int32_t ncuts, double *out)
{
    if (L < 1 || d < 1 || ncuts < 0) return -1;
    for (int32_t i = 0; i < ncuts; ++i) {
        if (cuts[i] <= 0 || cuts[i] >= L) return -1;
        if (i > 0 && cuts[i] <= cuts[i - 1]) return -1;
    }
    int32_t nchunks = ncuts + 1;
    double *m = (double *)malloc((size_t)nchunks * sizeof(double));
    double *l = (double *)malloc((size_t)nchunks * sizeof(double));
    double *acc = (double *)calloc((size_t)nchunks * (size_t)d, sizeof(double));
    if (!m || !l || !acc) { free(m); free(l); free(acc); return -2; }

    for (int32_t i = 0; i < nchunks; ++i) {
        int64_t j0 = (i == 0) ? 0 : cuts[i - 1];
        int64_t j1 = (i == ncuts) ? L : cuts[i];
        int64_t n = j1 - j0;
        double *s = (double *)malloc((size_t)n * sizeof(double));
        if (!s) { free(m); free(l); free(acc); return -2; }
        m[i] = -INFINITY;
        for (int64_t j = j0; j < j1; ++j) {
            double dot = 0.0;
            for (int32_t c = 0; c < d; ++c) dot += q[c] * K[j * d + c];
            s[j - j0] = scale * dot;
            if (s[j - j0] > m[i]) m[i] = s[j - j0];
        }
        l[i] = 0.0;
        for (int64_t j = j0; j < j1; ++j) {
            double w = exp(s[j - j0] - m[i]);
            l[i] += w;
            for (int32_t c = 0; c < d; ++c) acc[(size_t)i * d + c] += w * V[j * d + c];
        }
        free(s);
    }

    double mstar = -INFINITY;
    for (int32_t i = 0; i < nchunks; ++i) if (m[i] > mstar) mstar = m[i];
    double Z = 0.0;
    for (int32_t i = 0; i < nchunks; ++i) Z += l[i] * exp(m[i] - mstar);
    for (int32_t c = 0; c < d; ++c) {
        double o = 0.0;
        for (int32_t i = 0; i < nchunks; ++i) o += acc[(size_t)i * d + c] * exp(m[i] - mstar);
        out[c] = o / Z;
    }
    free(m); free(l); free(acc);
    return 0;
}

/* Element offset of (layer, page, kv head, K-or-V, slot, channel 0) in the pool format. */
static size_t pool_row_offset(int32_t num_pages, int32_t num_kv_heads, int32_t page_size,
                              int32_t head_dim, int32_t layer, int32_t page, int32_t kh,
                              int32_t k_or_v, int32_t slot)
{
    size_t o = (size_t)layer;
    o = o * (size_t)num_pages + (size_t)page;
    o = o * (size_t)num_kv_heads + (size_t)kh;
    o = o * 2u + (size_t)k_or_v;
    o = o * (size_t)page_size + (size_t)slot;
    return o * (size_t)head_dim;
}

/*
 * KV append: the token a request generates in this iteration has position L_r - 1 (seq_lens
 * hold the length AFTER the append).  Its key and value rows are copied, bit for bit, into
 * page block_tables[r][(L_r-1) / P], slot (L_r-1) % P, for every KV head.
 *   pool        bf16 bits, format above (modified in place)
 *   block_tables int32 [batch][max_pages_per_req]
 *   seq_lens    int32 [batch]
 *   k_new,v_new bf16 bits [batch][num_kv_heads][head_dim]
 * Returns 0; -1 if a length is < 1 or exceeds the table; -4 if a page id is out of range
 * (nothing is written for that request).
 */
int32_t oracle_kv_append(uint16_t *pool, int32_t num_layers, int32_t num_pages,
                         int32_t num_kv_heads, int32_t page_size, int32_t head_dim,
                         int32_t layer, int32_t batch, int32_t max_pages_per_req,
                         const int32_t *block_tables, const int32_t *seq_lens,
                         const uint16_t *k_new, const uint16_t *v_new)
{
    if (layer < 0 || layer >= num_layers) return -1;
    int32_t rc = 0;
    for (int32_t r = 0; r < batch; ++r) {
        int32_t L = seq_lens[r];
        if (L < 1 || (int64_t)L > (int64_t)max_pages_per_req * page_size) { rc = -1; continue; }
        int32_t pos = L - 1;
        int32_t page = block_tables[(size_t)r * max_pages_per_req + pos / page_size];
        int32_t slot = pos % page_size;
        if (page < 0 || page >= num_pages) { rc = -4; continue; }
        for (int32_t kh = 0; kh < num_kv_heads; ++kh) {
            size_t src = ((size_t)r * num_kv_heads + kh) * (size_t)head_dim;
            size_t dk = pool_row_offset(num_pages, num_kv_heads, page_size, head_dim,
                                        layer, page, kh, 0, slot);
            size_t dv = pool_row_offset(num_pages, num_kv_heads, page_size, head_dim,
                                        layer, page, kh, 1, slot);
            for (int32_t c = 0; c < head_dim; ++c) {
                pool[dk + c] = k_new[src + c];
                pool[dv + c] = v_new[src + c];
            }
        }
    }
    return rc;
}

/*
 * Paged grouped-query decode attention: for every request and KV head, gather the request's
 * L_r key and value rows in logical order through its block table, widen them to fp64, and
 * apply the dense definition once per query head of the group (kh = h / G, G = Hq / Hkv).
 *   q    bf16 bits [batch][num_q_heads][head_dim]
 *   out  fp64      [batch][num_q_heads][head_dim]   (not rounded)
 * scale = 1/sqrt(head_dim).  Returns 0; -1 bad length; -4 page id out of range (rows of that
 * request are left untouched).
 */
int32_t oracle_decode_attention(const uint16_t *pool, int32_t num_layers, int32_t num_pages,
                                int32_t num_q_heads, int32_t num_kv_heads, int32_t page_size,
                                int32_t head_dim, int32_t layer, int32_t batch,
                                int32_t max_pages_per_req, const int32_t *block_tables,
                                const int32_t *seq_lens, const uint16_t *q, double *out)
{
    if (layer < 0 || layer >= num_layers) return -1;
    if (num_kv_heads < 1 || num_q_heads % num_kv_heads != 0) return -1;
    const int32_t G = num_q_heads / num_kv_heads;
    const int32_t d = head_dim;
    const double scale = 1.0 / sqrt((double)d);
    int32_t rc = 0;

    /* validate first, so the parallel loop has no early exits */
    for (int32_t r = 0; r < batch; ++r) {
        int32_t L = seq_lens[r];
        if (L < 1 || (int64_t)L > (int64_t)max_pages_per_req * page_size) return -1;
        int32_t np = (L + page_size - 1) / page_size;
        for (int32_t i = 0; i < np; ++i) {
            int32_t page = block_tables[(size_t)r * max_pages_per_req + i];
            if (page < 0 || page >= num_pages) return -4;
        }
    }

    const int64_t npairs = (int64_t)batch * num_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t pair = 0; pair < npairs; ++pair) {
        const int32_t r = (int32_t)(pair / num_kv_heads);
        const int32_t kh = (int32_t)(pair % num_kv_heads);
        const int64_t L = seq_lens[r];
        double *K = (double *)malloc((size_t)L * d * sizeof(double));
        double *V = (double *)malloc((size_t)L * d * sizeof(double));
        double *qd = (double *)malloc((size_t)d * sizeof(double));
        if (!K || !V || !qd) {
#pragma omp atomic write
            rc = -2;
            free(K); free(V); free(qd);
            continue;
        }
        for (int64_t j = 0; j < L; ++j) {
            int32_t page = block_tables[(size_t)r * max_pages_per_req + j / page_size];
            int32_t slot = (int32_t)(j % page_size);
            size_t ok = pool_row_offset(num_pages, num_kv_heads, page_size, d, layer, page, kh, 0, slot);
            size_t ov = pool_row_offset(num_pages, num_kv_heads, page_size, d, layer, page, kh, 1, slot);
            for (int32_t c = 0; c < d; ++c) {
                K[j * d + c] = bf16_bits_to_f64(pool[ok + c]);
                V[j * d + c] = bf16_bits_to_f64(pool[ov + c]);
            }
        }
        for (int32_t g = 0; g < G; ++g) {
            const int32_t h = kh * G + g;
            const size_t qo = ((size_t)r * num_q_heads + h) * (size_t)d;
            for (int32_t c = 0; c < d; ++c) qd[c] = bf16_bits_to_f64(q[qo + c]);
            oracle_attention_dense_f64(qd, K, V, L, d, scale, out + qo, NULL);
        }
        free(K); free(V); free(qd);
    }
    return rc;
}

/*
 * Multi-token step (speculative-decoding verification, chunked append: paper Section 4 lists
 * speculative decoding and chunked prefill among the optimizations an instance may run with;
 * Section 6 "Experiment Setup" evaluates with speculative decoding enabled).  Each request appends
 * q_len tokens in this iteration: positions L_r - q_len .. L_r - 1 (seq_lens again hold the length
 * AFTER the append).  New token i's key/value rows go to page block_tables[r][pos / P], slot
 * pos % P, pos = L_r - q_len + i.
 *   k_new, v_new  bf16 bits [batch][q_len][num_kv_heads][head_dim]
 * Returns 0; -1 bad length (L < q_len or beyond the table); -4 page id out of range.
 */
int32_t oracle_kv_append_multi(uint16_t *pool, int32_t num_layers, int32_t num_pages,
                               int32_t num_kv_heads, int32_t page_size, int32_t head_dim,
                               int32_t layer, int32_t batch, int32_t q_len, int32_t max_pages_per_req,
                               const int32_t *block_tables, const int32_t *seq_lens,
                               const uint16_t *k_new, const uint16_t *v_new)
{
    if (layer < 0 || layer >= num_layers || q_len < 1) return -1;
    int32_t rc = 0;
    for (int32_t r = 0; r < batch; ++r) {
        int32_t L = seq_lens[r];
        if (L < q_len || (int64_t)L > (int64_t)max_pages_per_req * page_size) { rc = -1; continue; }
        for (int32_t i = 0; i < q_len; ++i) {
            int32_t pos = L - q_len + i;
            int32_t page = block_tables[(size_t)r * max_pages_per_req + pos / page_size];
            int32_t slot = pos % page_size;
            if (page < 0 || page >= num_pages) { rc = -4; continue; }
            for (int32_t kh = 0; kh < num_kv_heads; ++kh) {
                size_t src = (((size_t)r * q_len + i) * num_kv_heads + kh) * (size_t)head_dim;
                size_t dk = pool_row_offset(num_pages, num_kv_heads, page_size, head_dim, layer, page, kh, 0, slot);
                size_t dv = pool_row_offset(num_pages, num_kv_heads, page_size, head_dim, layer, page, kh, 1, slot);
                for (int32_t c = 0; c < head_dim; ++c) {
                    pool[dk + c] = k_new[src + c];
                    pool[dv + c] = v_new[src + c];
                }
            }
        }
    }
    return rc;
}

/*
 * Causal attention of the q_len new tokens of every request: query token i (position
 * L_r - q_len + i) attends to tokens 0 .. L_r - q_len + i, i.e. to everything before it and to
 * itself, through the dense definition above.
 *   q    bf16 bits [batch][q_len][num_q_heads][head_dim]
 *   out  fp64      [batch][q_len][num_q_heads][head_dim]
 * Returns 0; -1 bad length; -4 page id out of range.
 */
int32_t oracle_decode_attention_multi(const uint16_t *pool, int32_t num_layers, int32_t num_pages,
                                      int32_t num_q_heads, int32_t num_kv_heads, int32_t page_size,
                                      int32_t head_dim, int32_t layer, int32_t batch, int32_t q_len,
                                      int32_t max_pages_per_req, const int32_t *block_tables,
                                      const int32_t *seq_lens, const uint16_t *q, double *out)
{
    if (layer < 0 || layer >= num_layers || q_len < 1) return -1;
    if (num_kv_heads < 1 || num_q_heads % num_kv_heads != 0) return -1;
    const int32_t G = num_q_heads / num_kv_heads;
    const int32_t d = head_dim;
    const double scale = 1.0 / sqrt((double)d);
    int32_t rc = 0;
    for (int32_t r = 0; r < batch; ++r) {
        int32_t L = seq_lens[r];
        if (L < q_len || (int64_t)L > (int64_t)max_pages_per_req * page_size) return -1;
        int32_t np = (L + page_size - 1) / page_size;
        for (int32_t i = 0; i < np; ++i) {
            int32_t page = block_tables[(size_t)r * max_pages_per_req + i];
            if (page < 0 || page >= num_pages) return -4;
        }
    }
    const int64_t npairs = (int64_t)batch * num_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t pair = 0; pair < npairs; ++pair) {
        const int32_t r = (int32_t)(pair / num_kv_heads);
        const int32_t kh = (int32_t)(pair % num_kv_heads);
        const int64_t L = seq_lens[r];
        double *K = (double *)malloc((size_t)L * d * sizeof(double));
        double *V = (double *)malloc((size_t)L * d * sizeof(double));
        double *qd = (double *)malloc((size_t)d * sizeof(double));
        if (!K || !V || !qd) {
#pragma omp atomic write
            rc = -2;
            free(K); free(V); free(qd);
            continue;
        }
        for (int64_t j = 0; j < L; ++j) {
            int32_t page = block_tables[(size_t)r * max_pages_per_req + j / page_size];
            int32_t slot = (int32_t)(j % page_size);
            size_t ok = pool_row_offset(num_pages, num_kv_heads, page_size, d, layer, page, kh, 0, slot);
            size_t ov = pool_row_offset(num_pages, num_kv_heads, page_size, d, layer, page, kh, 1, slot);
            for (int32_t c = 0; c < d; ++c) {
                K[j * d + c] = bf16_bits_to_f64(pool[ok + c]);
                V[j * d + c] = bf16_bits_to_f64(pool[ov + c]);
            }
        }
        for (int32_t i = 0; i < q_len; ++i) {
            const int64_t visible = L - q_len + 1 + i;          /* tokens 0 .. own position */
            for (int32_t g = 0; g < G; ++g) {
                const int32_t h = kh * G + g;
                const size_t qo = (((size_t)r * q_len + i) * num_q_heads + h) * (size_t)d;
                for (int32_t c = 0; c < d; ++c) qd[c] = bf16_bits_to_f64(q[qo + c]);
                oracle_attention_dense_f64(qd, K, V, visible, d, scale, out + qo, NULL);
            }
        }
        free(K); free(V); free(qd);
    }
    return rc;
}
