// Local batch-size autoscaler (include/chiron_autoscaler.h): Algorithm 1 of the paper and a
// closed-loop driver over a measured latency curve.  Host-only.
#include "chiron_autoscaler.h"

#include <algorithm>
#include <cmath>
#include <limits>
#include <new>

namespace {
constexpr int32_t kOk = 0, kInval = -1, kNoMem = -2;

bool config_ok(const ckv_autoscaler_config *c)
{
    return c && c->alpha > 0.0 && c->alpha <= 1.0 && c->itl_slo_us > 0.0 && c->min_bs >= 1.0 && c->max_bs >= c->min_bs &&
           (c->tbp_mode == CKV_TBP_AFTER_INCREASE || c->tbp_mode == CKV_TBP_LITERAL);
}

double clamp(double x, double lo, double hi) { return std::min(std::max(x, lo), hi); }
}  // namespace

struct ckv_autoscaler {
    ckv_autoscaler_config cfg;
    double max_bs;
    double prev_throughput;
    bool has_prev;
};

namespace {
double step(ckv_autoscaler &a, double itl_us, double throughput, double *bp_out)
{
    const double lbp = itl_us / a.cfg.itl_slo_us;
    double tbp = 0.0;
    if (a.has_prev) tbp = throughput > 0.0 ? a.prev_throughput / throughput : std::numeric_limits<double>::infinity();
    const double bp = std::max(lbp, tbp);
    double next;
    if (bp < 1.0)
        next = bp > 0.0 ? a.cfg.alpha * (1.0 / bp) * a.max_bs + (1.0 - a.cfg.alpha) * a.max_bs : a.cfg.max_bs;
    else
        next = a.max_bs / 2.0;
    next = clamp(next, a.cfg.min_bs, a.cfg.max_bs);
    // default: TBP asks whether the last INCREASE of the batch size paid off, so the baseline is kept
    // only across one; literal: the throughput of the update before, always
    a.has_prev = a.cfg.tbp_mode == CKV_TBP_LITERAL || next > a.max_bs;
    a.prev_throughput = throughput;
    a.max_bs = next;
    if (bp_out) *bp_out = bp;
    return a.max_bs;
}

double curve(int32_t n, const double *x, const double *y, double bs)
{
    if (n == 1 || bs <= x[0]) return y[0];
    int i = 1;
    while (i < n - 1 && bs > x[i]) ++i;
    return y[i - 1] + (y[i] - y[i - 1]) * (bs - x[i - 1]) / (x[i] - x[i - 1]);
}
}  // namespace

extern "C" {

int32_t local_autoscaler_instance_slo(const double *itl_slos_us, int32_t n, double *out_slo_us)
{
    if (!itl_slos_us || n < 1 || !out_slo_us) return kInval;
    double m = itl_slos_us[0];
    for (int32_t i = 1; i < n; ++i) m = std::min(m, itl_slos_us[i]);
    if (!(m > 0.0)) return kInval;
    *out_slo_us = m;
    return kOk;
}

int32_t local_autoscaler_create(const ckv_autoscaler_config *cfg, double initial_max_bs, ckv_autoscaler **out)
{
    if (!out) return kInval;
    *out = nullptr;
    if (!config_ok(cfg) || !(initial_max_bs >= 1.0)) return kInval;
    ckv_autoscaler *a = new (std::nothrow) ckv_autoscaler();
    if (!a) return kNoMem;
    a->cfg = *cfg;
    a->max_bs = clamp(initial_max_bs, cfg->min_bs, cfg->max_bs);
    a->prev_throughput = 0.0;
    a->has_prev = false;
    *out = a;
    return kOk;
}

int32_t local_autoscaler_destroy(ckv_autoscaler *a)
{
    if (!a) return kInval;
    delete a;
    return kOk;
}

int32_t local_autoscaler_update(ckv_autoscaler *a, double itl_us, double throughput, double *out_max_bs,
                                double *out_backpressure)
{
    if (!a || !out_max_bs || !(itl_us > 0.0) || std::isnan(throughput)) return kInval;
    *out_max_bs = step(*a, itl_us, throughput, out_backpressure);
    return kOk;
}

int32_t local_autoscaler_get(const ckv_autoscaler *a, double *out_max_bs)
{
    if (!a || !out_max_bs) return kInval;
    *out_max_bs = a->max_bs;
    return kOk;
}

int32_t local_autoscaler_simulate(const ckv_autoscaler_config *cfg, double initial_max_bs, int32_t n_points,
                                  const double *batch_sizes, const double *us_per_step, double extra_us,
                                  int32_t demand, int32_t iterations, double *out_max_bs, int32_t *out_batch,
                                  double *out_itl_us, double *out_backpressure)
{
    if (!config_ok(cfg) || !(initial_max_bs >= 1.0) || n_points < 1 || !batch_sizes || !us_per_step) return kInval;
    if (demand < 1 || iterations < 1 || extra_us < 0.0) return kInval;
    for (int32_t i = 0; i < n_points; ++i) {
        if (!(us_per_step[i] > 0.0) || !(batch_sizes[i] >= 1.0)) return kInval;
        if (i > 0 && !(batch_sizes[i] > batch_sizes[i - 1])) return kInval;
    }
    ckv_autoscaler a;
    a.cfg = *cfg;
    a.max_bs = clamp(initial_max_bs, cfg->min_bs, cfg->max_bs);
    a.prev_throughput = 0.0;
    a.has_prev = false;
    for (int32_t k = 0; k < iterations; ++k) {
        const int32_t bs = std::max<int32_t>(1, (int32_t)std::min<double>(std::floor(a.max_bs), (double)demand));
        const double itl = curve(n_points, batch_sizes, us_per_step, (double)bs) + extra_us;
        double bp = 0.0;
        const double next = step(a, itl, (double)bs / itl, &bp);
        if (out_max_bs) out_max_bs[k] = next;
        if (out_batch) out_batch[k] = bs;
        if (out_itl_us) out_itl_us[k] = itl;
        if (out_backpressure) out_backpressure[k] = bp;
    }
    return kOk;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Global autoscaler primitives (Section 5).
// ------------------------------------------------------------------------------------------
#include <vector>

namespace {
double wait_seconds(int32_t ahead, double mu, double sigma, double thr, double z)
{
    if (ahead <= 0) return 0.0;
    return ((double)ahead * mu + z * sigma * std::sqrt((double)ahead)) / thr;
}

int32_t bbp_of(const int32_t *counts, const double *deadlines, int32_t n, double mu, double sigma, double thr, double z)
{
    int32_t bbp = 0;
    long long ahead = 0;
    for (int32_t g = 0; g < n; ++g) {
        if (counts[g] <= 0) continue;
        if (wait_seconds((int32_t)(ahead + counts[g] - 1), mu, sigma, thr, z) > deadlines[g]) ++bbp;
        ahead += counts[g];
    }
    return bbp;
}
}  // namespace

extern "C" {

int32_t global_request_groups(const double *ttft_slos, int32_t n, int32_t k, int32_t *out_group, double *out_centroids)
{
    if (!ttft_slos || n < 1 || k < 1 || !out_group) return kInval;
    k = std::min(k, n);
    std::vector<double> sorted(ttft_slos, ttft_slos + n);
    std::sort(sorted.begin(), sorted.end());
    std::vector<double> cent(k), next(k);
    for (int32_t j = 0; j < k; ++j) cent[j] = sorted[std::min<long long>(n - 1, (long long)(2 * j + 1) * n / (2 * k))];
    std::vector<int32_t> assign(n, 0), cur(n);
    for (int it = 0; it < 100; ++it) {
        for (int32_t i = 0; i < n; ++i) {
            int32_t best = 0;
            double bd = std::fabs(ttft_slos[i] - cent[0]);
            for (int32_t j = 1; j < k; ++j) {
                const double d = std::fabs(ttft_slos[i] - cent[j]);
                if (d < bd) { bd = d; best = j; }
            }
            cur[i] = best;
        }
        for (int32_t j = 0; j < k; ++j) {
            double sum = 0.0;
            long long cnt = 0;
            for (int32_t i = 0; i < n; ++i) if (cur[i] == j) { sum += ttft_slos[i]; ++cnt; }
            next[j] = cnt ? sum / (double)cnt : cent[j];
        }
        const bool fixed = (cur == assign) && (next == cent);
        assign = cur;
        cent = next;
        if (fixed) break;
    }
    std::vector<int32_t> rank(k);
    for (int32_t j = 0; j < k; ++j) rank[j] = j;
    std::stable_sort(rank.begin(), rank.end(), [&](int32_t a, int32_t b) { return cent[a] < cent[b]; });
    std::vector<int32_t> relabel(k);
    for (int32_t r = 0; r < k; ++r) relabel[rank[r]] = r;
    for (int32_t i = 0; i < n; ++i) out_group[i] = relabel[assign[i]];
    if (out_centroids) for (int32_t r = 0; r < k; ++r) out_centroids[r] = cent[rank[r]];
    return kOk;
}

int32_t global_waiting_time(int32_t requests_ahead, double mu_o, double sigma_o, double throughput, double z,
                            double *out_seconds)
{
    if (!out_seconds || !(throughput > 0.0) || mu_o < 0.0 || sigma_o < 0.0 || requests_ahead < 0) return kInval;
    *out_seconds = wait_seconds(requests_ahead, mu_o, sigma_o, throughput, z);
    return kOk;
}

int32_t global_batch_backpressure(const int32_t *counts, const double *deadlines, int32_t n_groups, double mu_o,
                                  double sigma_o, double throughput_per_instance, int32_t instances, double z,
                                  int32_t *out_bbp)
{
    if (!counts || !deadlines || n_groups < 0 || !out_bbp || instances < 1 || !(throughput_per_instance > 0.0)) return kInval;
    *out_bbp = bbp_of(counts, deadlines, n_groups, mu_o, sigma_o, throughput_per_instance * instances, z);
    return kOk;
}

int32_t global_batch_autoscale(const int32_t *counts, const double *deadlines, int32_t n_groups, double mu_o,
                               double sigma_o, double throughput_per_instance, int32_t current_instances,
                               int32_t active_requests, int32_t max_instances, double z, int32_t *out_instances)
{
    if (!out_instances || n_groups < 0 || (n_groups > 0 && (!counts || !deadlines))) return kInval;
    if (current_instances < 0 || active_requests < 0 || max_instances < 1 || !(throughput_per_instance > 0.0)) return kInval;
    long long queued = 0;
    for (int32_t g = 0; g < n_groups; ++g) queued += std::max(0, counts[g]);
    if (queued == 0) {
        *out_instances = active_requests == 0 ? 0 : current_instances;
        return kOk;
    }
    int32_t n = std::max(1, current_instances);
    while (n < max_instances && bbp_of(counts, deadlines, n_groups, mu_o, sigma_o, throughput_per_instance * n, z) > 0) ++n;
    *out_instances = n;
    return kOk;
}

int32_t global_interactive_autoscale(int32_t busy, int32_t total, double theta, double delta, int32_t floor_instances,
                                     int32_t *out_total)
{
    if (!out_total || busy < 0 || total < 0 || !(theta > 0.0) || theta > 1.0 || delta < 0.0 || floor_instances < 0) return kInval;
    total = std::max(std::max(total, floor_instances), 1);
    const double ibp = (double)busy / (double)total;
    if (ibp >= theta - delta && ibp <= theta + delta) { *out_total = total; return kOk; }
    const int32_t want = (int32_t)std::ceil((double)busy / theta - 1e-12);
    *out_total = std::max(std::max(floor_instances, busy), want);
    return kOk;
}

}  // extern "C"
