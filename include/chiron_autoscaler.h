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
    int32_t tbp_mode;    /* CKV_TBP_AFTER_INCREASE (default) or CKV_TBP_LITERAL, see local_autoscaler_update */
} ckv_autoscaler_config;

#define CKV_TBP_AFTER_INCREASE 0
#define CKV_TBP_LITERAL        1

typedef struct ckv_autoscaler ckv_autoscaler;   /* host object: MaxBS and the previous throughput */

/* Smallest ITL SLO of a set of requests: the SLO an instance is held to (Section 4.2, closing
 * remark).  n >= 1. */
int32_t local_autoscaler_instance_slo(const double *itl_slos_us, int32_t n, double *out_slo_us);

int32_t local_autoscaler_create(const ckv_autoscaler_config *cfg, double initial_max_bs, ckv_autoscaler **out);
int32_t local_autoscaler_destroy(ckv_autoscaler *a);

/*
 * One pass of Algorithm 1's update loop ("for each change in the GPU running queue"):
 *   LBP = itl / ITL SLO;  TBP = previous throughput / current throughput (0 if there is none);
 *   BP = max(LBP, TBP);   BP < 1: MaxBS <- alpha*(1/BP)*MaxBS + (1-alpha)*MaxBS;  else MaxBS <- MaxBS/2
 * then clamped to [min_bs, max_bs].  A backpressure of exactly 1 halves.  itl_us > 0; a
 * throughput <= 0 counts as infinite backpressure.
 * Which throughput is "previous" (Algorithm 1 prints TBP = Throughput_prev / Throughput_curr):
 *   CKV_TBP_LITERAL         the throughput of the update before, whatever that update did;
 *   CKV_TBP_AFTER_INCREASE  that throughput only if the update before INCREASED MaxBS -- Section
 *                           4.1 introduces TBP as the test whether raising the batch size still
 *                           pays -- and none (TBP = 0) after a decrease.
 * The literal rule is unstable in closed loop on the rising part of a throughput curve: a halving
 * lowers the throughput, the next update reads TBP > 1 and halves again, down to min_bs.  The
 * default avoids that; the literal rule is kept for comparison.
 * out_backpressure may be NULL.
 */
int32_t local_autoscaler_update(ckv_autoscaler *a, double itl_us, double throughput, double *out_max_bs,
                                double *out_backpressure);

/* Current maximum batch size. */
int32_t local_autoscaler_get(const ckv_autoscaler *a, double *out_max_bs);

/*
 * Closed loop against a measured latency curve (the ITL / throughput against batch size figure of
 * Section 2.1): at every iteration the instance
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

/* ------------------------------------------------------------------------------------------
 * The global autoscaler in time: a discrete-event simulation of Section 3 (life cycle of a
 * request, instance classes, routing, eviction from mixed instances) driven by Section 5
 * (interactive autoscaling on the IBP band, batch autoscaling by Algorithm 2 on request groups
 * and the waiting-time estimate of Eq. 1).  Host-only and deterministic: every random quantity
 * (arrival times, output lengths) is an INPUT.
 *
 * Model.  An instance has a class -- interactive, mixed or batch -- a number of slots (its
 * maximum batch size, which the local autoscaler of Section 4 would hold it at) and a token rate
 * per running request (1 / ITL at that batch size); interactive and mixed instances share one
 * (slots, rate) pair because a mixed instance is sized by the interactive ITL SLO (Section 2.3).
 * A request with O output tokens occupies one slot for O / rate seconds; prefill is not modelled,
 * so TTFT = first start - arrival.  A new instance is usable startup_s after it was added.
 *
 * Rules (each applied in exactly this order, so that two implementations produce the same event
 * sequence):
 *  - Events are handled in order of time; at equal times: request completions (by request id),
 *    instances becoming ready (by instance id), arrivals (by request id), then the autoscaler
 *    tick.  Ticks fall at k * tick_s, k = 1, 2, ...  After every event pending work is dispatched.
 *  - Interactive arrival (zero queuing, Section 5.3 footnote): the lowest-numbered ready
 *    interactive instance with a free slot; else the lowest-numbered ready mixed instance with a
 *    free slot; else the lowest-numbered ready mixed instance that runs a batch request, whose
 *    most recently started batch request (ties: higher request id) is evicted -- it returns to
 *    the global queue with the tokens it still has to produce (its KV cache was saved, Section
 *    3) and its original arrival time.  If none of these exists the request waits, first come
 *    first served, and is placed as soon as a dispatch finds room.
 *  - Batch arrival: the request joins the global queue.  Queue order: request group (increasing
 *    TTFT SLO centroid), then arrival time, then id.  Groups are re-formed at every tick
 *    (global_request_groups over the queued requests, groups_k groups); a request that arrives
 *    between ticks takes the group with the nearest centroid (ties: the lower; no centroid yet:
 *    group 0).
 *  - Dispatch: waiting interactive requests first.  Then, while the queue is not empty: the
 *    lowest-numbered ready batch instance with a free slot, else -- if no interactive request
 *    is waiting -- the lowest-numbered ready mixed instance with a free slot, takes the head of
 *    the queue.
 *  - Tick, interactive side (Section 5.2): busy = ready interactive or mixed instances that run
 *    at least one interactive request, total = interactive + mixed instances not yet removed
 *    (starting ones included, which is what stops the growth while they load); target =
 *    global_interactive_autoscale(busy, total, theta, delta, floor_instances).  target > total
 *    adds instances: interactive ones until their number reaches max(1, floor(theta * target +
 *    1/2)), mixed ones after that.  target < total removes instances that run no interactive
 *    request, in this order: still starting before ready, mixed before interactive, higher id
 *    first; batch requests on a removed instance are evicted to the queue.
 *  - Tick, batch side (Section 5.3, Algorithm 2), policy CKV_SIM_POLICY_CHIRON: with G groups in
 *    queue order, counts[g] requests and deadline[g] = min over the group of (arrival + TTFT
 *    SLO) - now, a group is late at n batch instances if its last request's estimated wait
 *        W_g = (a mu_o + z sigma_o sqrt(a)) / (n (slots_batch rate_batch) + spare),
 *        a = requests in earlier groups + counts[g] - 1,
 *    exceeds deadline[g]; spare = rate_interactive x free slots on ready mixed instances (the
 *    over-provisioned capacity batch requests may use); with no throughput at all every
 *    non-empty group is late.  (mu_o, sigma_o) are the running mean and sample deviation of the
 *    output lengths of completed requests, the priors until two have completed.  If some group
 *    is late at the current count n (starting ones included), n grows by one until none is or
 *    max_batch_instances is reached, and the difference is added.  If the queue is empty and no
 *    request runs on a batch instance, all batch instances are removed.
 *  - Policy CKV_SIM_POLICY_IMMEDIATE is the contrast of Section 2.3 ("immediate autoscaling"):
 *    no batch autoscaling at ticks; a batch arrival that is still queued after dispatch adds
 *    one batch instance unless the starting ones already have slots for the whole queue, and a
 *    batch instance that runs nothing after the dispatch that follows a completion on it is
 *    removed at once.
 *  - The run ends when every request has completed (or at horizon_s, if > 0).
 *
 * Arithmetic that decides event times (both sides must use exactly these expressions):
 *   finish = start + remaining / rate;   on eviction remaining = max(remaining - (now - start) * rate, 0).
 */
#define CKV_SIM_POLICY_CHIRON    0
#define CKV_SIM_POLICY_IMMEDIATE 1

#define CKV_SIM_EV_ARRIVE 0   /* a = request                       b = -1                      */
#define CKV_SIM_EV_START  1   /* a = request                       b = instance                */
#define CKV_SIM_EV_EVICT  2   /* a = request                       b = instance                */
#define CKV_SIM_EV_FINISH 3   /* a = request                       b = instance                */
#define CKV_SIM_EV_ADD    4   /* a = instance                      b = class (0 int, 1 mixed, 2 batch) */
#define CKV_SIM_EV_READY  5   /* a = instance                      b = class                   */
#define CKV_SIM_EV_REMOVE 6   /* a = instance                      b = class                   */
#define CKV_SIM_EV_TICK   7   /* a = interactive + mixed instances b = batch instances (after the tick) */

typedef struct ckv_sim_config {
    int32_t slots_interactive;    /* max batch size of interactive and mixed instances */
    int32_t slots_batch;          /* max batch size of batch instances */
    double rate_interactive;      /* output tokens per second of one running request there */
    double rate_batch;
    double startup_s;             /* model load time of a new instance (Section 2.3: 15 s to a minute) */
    double tick_s;                /* period of the global autoscaler */
    double theta, delta;          /* IBP band (Section 5.2) */
    int32_t floor_instances;      /* interactive + mixed instances never drop below this */
    int32_t initial_instances;    /* interactive + mixed instances ready at time 0 */
    int32_t max_batch_instances;
    int32_t groups_k;             /* request groups formed from the queue */
    double z;                     /* quantile of the waiting-time estimate (0: the mean, Eq. 1) */
    double mu_o_prior, sigma_o_prior;
    int32_t policy;               /* CKV_SIM_POLICY_* */
    double horizon_s;             /* stop here even if requests remain; <= 0: run to completion */
} ckv_sim_config;

typedef struct ckv_sim_summary {
    double end_s;                       /* time of the last handled event */
    int32_t finished;                   /* requests completed */
    int32_t interactive_total, interactive_ttft_met;
    int32_t batch_total, batch_ttft_met;   /* met: started within the TTFT SLO */
    int32_t evictions;
    int32_t instances_added[3], instances_removed[3];   /* per class; the initial instances are not counted */
    double instance_seconds[3];         /* per class, from the add (start-up included) to the removal or the end */
    int32_t peak_instances[3];
    double tokens_served;
} ckv_sim_summary;

/*
 * Run the simulation.  Requests i = 0 .. n-1 are given in order of arrival (arrival_s
 * non-decreasing): kind[i] 0 = interactive, 1 = batch; output_tokens[i] >= 1; ttft_slo_s[i] > 0.
 * Outputs (any may be NULL): per request the time of its first start (-1 if it never started),
 * its completion time (-1 if it did not complete) and how often it was evicted; the summary; and
 * the event log: row r is (log_time[r], log_rows[3r] = CKV_SIM_EV_*, log_rows[3r+1] = a,
 * log_rows[3r+2] = b), at most log_cap rows are written, *out_log_rows receives the number of
 * events that occurred.  Errors: CKV_EINVAL (configuration or inputs), CKV_ENOMEM.
 */
int32_t global_autoscaler_simulate(const ckv_sim_config *cfg, int32_t n, const double *arrival_s,
                                   const int32_t *kind, const double *output_tokens, const double *ttft_slo_s,
                                   double *out_first_start_s, double *out_finish_s, int32_t *out_evictions,
                                   ckv_sim_summary *out_summary, double *log_time, int32_t *log_rows,
                                   int32_t log_cap, int64_t *out_log_rows);

#ifdef __cplusplus
}
#endif
#endif /* CHIRON_AUTOSCALER_H */
