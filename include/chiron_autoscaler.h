/*
 * chiron_autoscaler.h -- C ABI of the local (per-instance) batch-size autoscaler: the consumer of
 * the latency-versus-batch-size curve that step_latency_sweep (chiron_kv.h) measures.
 *
 * Paper: Section 4 "Local Autoscaler"; backpressure definitions in Section 4.1 "Local
 * Backpressure"; the update rule is Algorithm 1 (Section 4.2 "Batch Size Autoscaling").
 * Host-only code: no CUDA call, no device memory.
 *
 * All functions return CKV_OK (0) or a negative code (CKV_EINVAL on bad arguments).
 */
#ifndef CHIRON_AUTOSCALER_H
#define CHIRON_AUTOSCALER_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ckv_autoscaler_config {
    double alpha;        /* EWMA smoothing factor of Algorithm 1 (the paper uses 0.5); 0 < alpha <= 1 */
    double itl_slo_us;   /* the instance's ITL SLO: the smallest ITL SLO among its requests (Section 4.2) */
    double min_bs;       /* lower clamp of the maximum batch size, >= 1 */
    double max_bs;       /* upper clamp of the maximum batch size */
} ckv_autoscaler_config;

typedef struct ckv_autoscaler ckv_autoscaler;   /* host object: MaxBS and the previous throughput */

/* Smallest ITL SLO of a set of requests (Section 4.2: "the ITL SLO for the instance is the smallest
 * ITL SLO amongst all requests executing on that instance").  n >= 1. */
int32_t local_autoscaler_instance_slo(const double *itl_slos_us, int32_t n, double *out_slo_us);

int32_t local_autoscaler_create(const ckv_autoscaler_config *cfg, double initial_max_bs, ckv_autoscaler **out);
int32_t local_autoscaler_destroy(ckv_autoscaler *a);

/*
 * One pass of Algorithm 1's update loop ("for each change in the GPU running queue"):
 *   LBP = itl / ITL SLO;  TBP = previous throughput / current throughput (0 if there is none);
 *   BP = max(LBP, TBP);   BP < 1: MaxBS <- alpha*(1/BP)*MaxBS + (1-alpha)*MaxBS;  else MaxBS <- MaxBS/2
 * then clamped to [min_bs, max_bs].  A backpressure of exactly 1 halves.  itl_us > 0; a
 * throughput <= 0 counts as infinite backpressure.  The previous throughput is remembered only
 * across an update that increased MaxBS (Section 4.1: TBP > 1 means "no throughput gain is
 * observed from increasing the batch size"); after a decrease TBP is 0 for one update -- otherwise
 * every halving lowers the throughput, reads as TBP > 1 and triggers the next halving.
 * out_backpressure may be NULL.
 */
int32_t local_autoscaler_update(ckv_autoscaler *a, double itl_us, double throughput, double *out_max_bs,
                                double *out_backpressure);

/* Current maximum batch size. */
int32_t local_autoscaler_get(const ckv_autoscaler *a, double *out_max_bs);

/*
 * Closed loop against a measured latency curve (Section 2.1 figure "Variation in inter-token
 * latency and token throughput with increasing batch size"): at every iteration the instance
 * runs batch = min(floor(MaxBS), demand), observes ITL = curve(batch) + extra_us (curve: linear
 * interpolation of (batch_sizes[i], us_per_step[i]), n_points >= 1, batch sizes increasing; the
 * last slope continues beyond the last point; extra_us stands for everything outside attention,
 * e.g. weight streaming) and throughput = batch / ITL, and applies local_autoscaler_update.
 * Outputs, each [iterations] (any may be NULL): MaxBS after the update, batch run, ITL, backpressure.
 */
int32_t local_autoscaler_simulate(const ckv_autoscaler_config *cfg, double initial_max_bs,
                                  int32_t n_points, const double *batch_sizes, const double *us_per_step,
                                  double extra_us, int32_t demand, int32_t iterations,
                                  double *out_max_bs, int32_t *out_batch, double *out_itl_us,
                                  double *out_backpressure);

#ifdef __cplusplus
}
#endif
#endif /* CHIRON_AUTOSCALER_H */
