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

/* ------------------------------------------------------------------------------------------
 * Global autoscaler primitives (Section 5 "Global Autoscaler").  Host-only.
 * ------------------------------------------------------------------------------------------ */

/*
 * Request groups (Section 5.3, "Request Group Creation"): cluster the queued requests by TTFT SLO
 * with 1-D k-means.  Centroids start at evenly spaced quantiles of the sorted values and Lloyd
 * iterations run to a fixed point (at most 100); groups are numbered by increasing centroid, ties
 * in distance go to the lower centroid.  k is clamped to [1, n].
 *   out_group [n]: group of every request;  out_centroids [k] (may be NULL).
 */
int32_t global_request_groups(const double *ttft_slos, int32_t n, int32_t k, int32_t *out_group,
                              double *out_centroids);

/*
 * Waiting time of a request with `requests_ahead` requests before it in the queue (Eq. 1): the
 * output tokens ahead are a sum of i.i.d. lengths with fitted mean mu_o and deviation sigma_o
 * (normal by the CLT), served at a constant token throughput:
 *   W = (requests_ahead * mu_o + z * sigma_o * sqrt(requests_ahead)) / throughput
 * z = 0 gives the mean estimate; z > 0 a conservative quantile.
 */
int32_t global_waiting_time(int32_t requests_ahead, double mu_o, double sigma_o, double throughput, double z,
                            double *out_seconds);

/*
 * Batch backpressure (Section 5.3): BBP = number of request groups whose estimated waiting time
 * exceeds their TTFT deadline.  Groups are given in service order (increasing TTFT SLO, FCFS
 * inside); group g's waiting time is that of its LAST request: requests_ahead = requests of the
 * earlier groups + counts[g] - 1, at throughput_per_instance * instances.  deadlines[g] is the
 * time the group still has (its TTFT SLO minus the age of its oldest request).
 */
int32_t global_batch_backpressure(const int32_t *counts, const double *deadlines, int32_t n_groups, double mu_o,
                                  double sigma_o, double throughput_per_instance, int32_t instances, double z,
                                  int32_t *out_bbp);

/*
 * Algorithm 2 (Batch Instance Autoscaling): starting from the instances already dispatched (at
 * least one), add one instance at a time until BBP = 0 or max_instances is reached; with an empty
 * queue, retire every batch instance once no request is active on them.
 */
int32_t global_batch_autoscale(const int32_t *counts, const double *deadlines, int32_t n_groups, double mu_o,
                               double sigma_o, double throughput_per_instance, int32_t current_instances,
                               int32_t active_requests, int32_t max_instances, double z, int32_t *out_instances);

/*
 * Interactive autoscaling (Section 5.2): IBP = instances running interactive requests / (mixed +
 * interactive instances).  While IBP stays inside [theta - delta, theta + delta] the count is
 * kept; outside the band it becomes ceil(busy / theta), never below `busy` or `floor_instances`.
 */
int32_t global_interactive_autoscale(int32_t busy, int32_t total, double theta, double delta,
                                     int32_t floor_instances, int32_t *out_total);

#ifdef __cplusplus
}
#endif
#endif /* CHIRON_AUTOSCALER_H */
