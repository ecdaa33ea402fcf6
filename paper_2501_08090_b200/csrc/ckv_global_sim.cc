// The global autoscaler in time (include/chiron_autoscaler.h, global_autoscaler_simulate): a
// discrete-event simulation of the request life cycle of Section 3 under the autoscaling rules
// of Section 5.  Host-only.  The rules and their order are stated in the header; this file keeps
// the pending events in ordered containers (completions and instance start-ups in std::set,
// arrivals behind a cursor, the tick behind a counter) and picks the earliest at every step.
#include "chiron_autoscaler.h"

#include <algorithm>
#include <cmath>
#include <deque>
#include <limits>
#include <set>
#include <tuple>
#include <utility>
#include <vector>

namespace {

constexpr int32_t kOk = 0, kInval = -1, kNoMem = -2;
constexpr int kInteractive = 0, kMixed = 1, kBatch = 2;
constexpr double kNever = std::numeric_limits<double>::infinity();

struct Request {
    double arrival, tokens, slo;
    int kind;
    double remaining, start = -1.0, finish_at = -1.0;
    int inst = -1, group = 0, evictions = 0;
    double first_start = -1.0, finished_at = -1.0;
};

struct Instance {
    int cls;
    double added_at, ready_at;
    bool ready = false, removed = false;
    int n_interactive = 0;
    std::set<std::pair<double, int>> batch_running;      // (start time, request): the last one is the eviction victim
    int used() const { return n_interactive + (int)batch_running.size(); }
};

class Simulation {
public:
    Simulation(const ckv_sim_config &c, int32_t n, const double *arrival, const int32_t *kind, const double *tokens,
               const double *slo, double *log_time, int32_t *log_rows, int32_t log_cap)
        : cfg(c), log_time_(log_time), log_rows_(log_rows), log_cap_(log_cap)
    {
        reqs.resize(n);
        for (int32_t i = 0; i < n; ++i) {
            reqs[i].arrival = arrival[i]; reqs[i].tokens = tokens[i]; reqs[i].slo = slo[i]; reqs[i].kind = kind[i];
            reqs[i].remaining = tokens[i];
        }
        for (int i = 0; i < cfg.initial_instances; ++i) {
            const int want_int = std::max(1, (int)std::floor(cfg.theta * cfg.initial_instances + 0.5));
            const int id = new_instance((int)alive[kInteractive].size() < want_int ? kInteractive : kMixed, 0.0, false);
            insts[id].ready = true;
        }
    }

    void run()
    {
        const int n = (int)reqs.size();
        long long tick_k = 1;
        while (finished < n) {
            const double t_fin = finishes.empty() ? kNever : finishes.begin()->first;
            const double t_rdy = readies.empty() ? kNever : readies.begin()->first;
            const double t_arr = next_arrival < n ? reqs[next_arrival].arrival : kNever;
            const double t_tick = (double)tick_k * cfg.tick_s;
            // earliest first; at equal times completions, start-ups, arrivals, tick
            int which = 3;
            double t = t_tick;
            if (t_arr <= t) { which = 2; t = t_arr; }
            if (t_rdy <= t) { which = 1; t = t_rdy; }
            if (t_fin <= t) { which = 0; t = t_fin; }
            if (cfg.horizon_s > 0.0 && t > cfg.horizon_s) break;
            now = t;
            if (which == 0) {
                on_finish(finishes.begin()->second);
            } else if (which == 1) {
                const int id = readies.begin()->second;
                readies.erase(readies.begin());
                insts[id].ready = true;
                log(CKV_SIM_EV_READY, id, insts[id].cls);
                dispatch();
            } else if (which == 2) {
                on_arrival(next_arrival++);
            } else {
                const long long added_before = total_added;
                on_tick();
                ++tick_k;
                // nothing runs, nothing starts, nothing will arrive and the tick added nothing: stuck
                if (finishes.empty() && readies.empty() && next_arrival == n && total_added == added_before) break;
            }
            if (events > 400000000ll) break;
        }
        end = now;
        for (auto &in : insts)
            if (!in.removed) seconds[in.cls] += end - in.added_at;
    }

    void summary(ckv_sim_summary *s) const
    {
        *s = ckv_sim_summary{};
        s->end_s = end;
        s->finished = finished;
        for (const Request &r : reqs) {
            const bool met = r.first_start >= 0.0 && r.first_start - r.arrival <= r.slo;
            if (r.kind == 0) { ++s->interactive_total; s->interactive_ttft_met += met; }
            else { ++s->batch_total; s->batch_ttft_met += met; }
            s->evictions += r.evictions;
        }
        for (int c = 0; c < 3; ++c) {
            s->instances_added[c] = added[c]; s->instances_removed[c] = removed[c];
            s->instance_seconds[c] = seconds[c]; s->peak_instances[c] = peak[c];
        }
        s->tokens_served = tokens_served;
    }

    std::vector<Request> reqs;
    long long events = 0;

private:
    const ckv_sim_config cfg;
    std::vector<Instance> insts;
    std::set<int> alive[3];                                       // instances not removed, by class
    std::set<std::pair<double, int>> finishes, readies;           // (time, request) / (time, instance)
    std::set<std::tuple<int, double, int>> queue;                 // (group, arrival, request)
    std::deque<int> waiting;                                      // interactive requests without a slot
    std::vector<double> centroids;
    int next_arrival = 0, finished = 0;
    double now = 0.0, end = 0.0;
    long long total_added = 0;
    int added[3] = {0, 0, 0}, removed[3] = {0, 0, 0}, peak[3] = {0, 0, 0};
    double seconds[3] = {0.0, 0.0, 0.0}, tokens_served = 0.0;
    long long fit_n = 0;
    double fit_mean = 0.0, fit_m2 = 0.0;
    double *log_time_;
    int32_t *log_rows_;
    int32_t log_cap_;

    void log(int kind, int a, int b)
    {
        if (log_time_ && log_rows_ && events < log_cap_) {
            log_time_[events] = now;
            log_rows_[3 * events] = kind; log_rows_[3 * events + 1] = a; log_rows_[3 * events + 2] = b;
        }
        ++events;
    }

    double rate_of(int cls) const { return cls == kBatch ? cfg.rate_batch : cfg.rate_interactive; }
    int slots_of(int cls) const { return cls == kBatch ? cfg.slots_batch : cfg.slots_interactive; }

    int new_instance(int cls, double ready_at, bool counted)
    {
        Instance in;
        in.cls = cls; in.added_at = now; in.ready_at = ready_at;
        insts.push_back(in);
        const int id = (int)insts.size() - 1;
        alive[cls].insert(id);
        peak[cls] = std::max(peak[cls], (int)alive[cls].size());
        if (counted) {
            ++added[cls]; ++total_added;
            readies.insert({ready_at, id});
            log(CKV_SIM_EV_ADD, id, cls);
        }
        return id;
    }

    void remove_instance(int id)
    {
        Instance &in = insts[id];
        std::vector<int> victims;
        for (auto &e : in.batch_running) victims.push_back(e.second);
        std::sort(victims.begin(), victims.end());
        for (int r : victims) evict(r);
        if (!in.ready) readies.erase({in.ready_at, id});
        in.removed = true;
        alive[in.cls].erase(id);
        ++removed[in.cls];
        seconds[in.cls] += now - in.added_at;
        log(CKV_SIM_EV_REMOVE, id, in.cls);
    }

    int group_of(double slo) const
    {
        int best = 0;
        for (int j = 1; j < (int)centroids.size(); ++j)
            if (std::fabs(slo - centroids[j]) < std::fabs(slo - centroids[best])) best = j;
        return best;
    }

    void enqueue(int r)
    {
        reqs[r].group = group_of(reqs[r].slo);
        queue.insert(std::make_tuple(reqs[r].group, reqs[r].arrival, r));
    }

    void start(int r, int id)
    {
        Request &q = reqs[r];
        Instance &in = insts[id];
        q.inst = id; q.start = now;
        if (q.first_start < 0.0) q.first_start = now;
        q.finish_at = now + q.remaining / rate_of(in.cls);
        finishes.insert({q.finish_at, r});
        if (q.kind == 0) ++in.n_interactive; else in.batch_running.insert({now, r});
        log(CKV_SIM_EV_START, r, id);
    }

    void evict(int r)
    {
        Request &q = reqs[r];
        Instance &in = insts[q.inst];
        q.remaining = std::max(q.remaining - (now - q.start) * rate_of(in.cls), 0.0);
        finishes.erase({q.finish_at, r});
        in.batch_running.erase({q.start, r});
        log(CKV_SIM_EV_EVICT, r, q.inst);
        q.inst = -1;
        ++q.evictions;
        enqueue(r);
    }

    int first_with_room(int cls) const
    {
        for (int id : alive[cls])
            if (insts[id].ready && insts[id].used() < slots_of(cls)) return id;
        return -1;
    }

    bool place_interactive(int r)
    {
        int id = first_with_room(kInteractive);
        if (id < 0) id = first_with_room(kMixed);
        if (id < 0) {
            for (int m : alive[kMixed]) {
                if (insts[m].ready && !insts[m].batch_running.empty()) {
                    evict(insts[m].batch_running.rbegin()->second);
                    id = m;
                    break;
                }
            }
        }
        if (id < 0) return false;
        start(r, id);
        return true;
    }

    void dispatch()
    {
        while (!waiting.empty() && place_interactive(waiting.front())) waiting.pop_front();
        while (!queue.empty()) {
            int id = first_with_room(kBatch);
            if (id < 0 && waiting.empty()) id = first_with_room(kMixed);
            if (id < 0) break;
            const int r = std::get<2>(*queue.begin());
            queue.erase(queue.begin());
            start(r, id);
        }
    }

    void on_arrival(int r)
    {
        log(CKV_SIM_EV_ARRIVE, r, -1);
        if (reqs[r].kind == 0) {
            if (!waiting.empty() || !place_interactive(r)) waiting.push_back(r);
            dispatch();
            return;
        }
        enqueue(r);
        dispatch();
        if (cfg.policy == CKV_SIM_POLICY_IMMEDIATE && reqs[r].inst < 0) {
            long long promised = 0;
            for (int id : alive[kBatch])
                if (!insts[id].ready) promised += cfg.slots_batch;
            if ((long long)queue.size() > promised && (int)alive[kBatch].size() < cfg.max_batch_instances)
                new_instance(kBatch, now + cfg.startup_s, true);
        }
    }

    void on_finish(int r)
    {
        Request &q = reqs[r];
        Instance &in = insts[q.inst];
        const int id = q.inst;
        finishes.erase({q.finish_at, r});
        if (q.kind == 0) --in.n_interactive; else in.batch_running.erase({q.start, r});
        q.finished_at = now; q.remaining = 0.0; q.inst = -1;
        ++finished;
        tokens_served += q.tokens;
        ++fit_n;                                                  // running fit of the output lengths
        const double d = q.tokens - fit_mean;
        fit_mean += d / (double)fit_n;
        fit_m2 += d * (q.tokens - fit_mean);
        log(CKV_SIM_EV_FINISH, r, id);
        dispatch();
        if (cfg.policy == CKV_SIM_POLICY_IMMEDIATE && in.cls == kBatch && in.used() == 0) remove_instance(id);
    }

    void regroup()
    {
        std::vector<int> ids;
        std::vector<double> slos;
        for (auto &e : queue) { ids.push_back(std::get<2>(e)); slos.push_back(reqs[std::get<2>(e)].slo); }
        queue.clear();
        centroids.clear();
        if (ids.empty()) return;
        const int n = (int)ids.size(), k = std::max(1, std::min(cfg.groups_k, n));
        std::vector<int32_t> grp(n);
        centroids.resize(k);
        global_request_groups(slos.data(), n, k, grp.data(), centroids.data());
        for (int i = 0; i < n; ++i) {
            reqs[ids[i]].group = grp[i];
            queue.insert(std::make_tuple((int)grp[i], reqs[ids[i]].arrival, ids[i]));
        }
    }

    void scale_interactive()
    {
        int busy = 0;
        for (int c = kInteractive; c <= kMixed; ++c)
            for (int id : alive[c])
                if (insts[id].ready && insts[id].n_interactive > 0) ++busy;
        const int total = (int)(alive[kInteractive].size() + alive[kMixed].size());
        int32_t target = total;
        global_interactive_autoscale(busy, total, cfg.theta, cfg.delta, cfg.floor_instances, &target);
        if (target > total) {
            const int want_int = std::max(1, (int)std::floor(cfg.theta * target + 0.5));
            for (int i = total; i < target; ++i)
                new_instance((int)alive[kInteractive].size() < want_int ? kInteractive : kMixed, now + cfg.startup_s, true);
        } else if (target < total) {
            std::vector<std::tuple<int, int, int>> cand;          // (ready, interactive class, -id)
            for (int c = kInteractive; c <= kMixed; ++c)
                for (int id : alive[c])
                    if (insts[id].n_interactive == 0) cand.push_back(std::make_tuple(insts[id].ready ? 1 : 0, c == kInteractive ? 1 : 0, -id));
            std::sort(cand.begin(), cand.end());
            for (int i = 0; i < (int)cand.size() && i < total - target; ++i) remove_instance(-std::get<2>(cand[i]));
        }
    }

    void scale_batch()
    {
        if (queue.empty()) {
            int active = 0;
            for (int id : alive[kBatch]) active += insts[id].used();
            if (active == 0) {
                const std::vector<int> ids(alive[kBatch].begin(), alive[kBatch].end());
                for (int id : ids) remove_instance(id);
            }
            return;
        }
        std::vector<double> counts, deadlines;                    // per non-empty group, in queue order
        int cur = -1;
        for (auto &e : queue) {
            const Request &q = reqs[std::get<2>(e)];
            if (std::get<0>(e) != cur) { cur = std::get<0>(e); counts.push_back(0.0); deadlines.push_back(kNever); }
            counts.back() += 1.0;
            deadlines.back() = std::min(deadlines.back(), q.arrival + q.slo - now);
        }
        double spare = 0.0;
        for (int id : alive[kMixed])
            if (insts[id].ready) spare += cfg.rate_interactive * (double)(cfg.slots_interactive - insts[id].used());
        const double mu = fit_n >= 2 ? fit_mean : cfg.mu_o_prior;
        const double sigma = fit_n >= 2 ? std::sqrt(fit_m2 / (double)(fit_n - 1)) : cfg.sigma_o_prior;
        auto late = [&](int n) {
            const double thr = (double)n * ((double)cfg.slots_batch * cfg.rate_batch) + spare;
            double ahead = 0.0;
            for (size_t g = 0; g < counts.size(); ++g) {
                const double a = ahead + counts[g] - 1.0;
                if (!(thr > 0.0)) return true;
                if ((a * mu + cfg.z * sigma * std::sqrt(a)) / thr > deadlines[g]) return true;
                ahead += counts[g];
            }
            return false;
        };
        const int n_cur = (int)alive[kBatch].size();
        int n = n_cur;
        while (n < cfg.max_batch_instances && late(n)) ++n;
        for (int i = n_cur; i < n; ++i) new_instance(kBatch, now + cfg.startup_s, true);
    }

    void on_tick()
    {
        regroup();
        scale_interactive();
        if (cfg.policy == CKV_SIM_POLICY_CHIRON) scale_batch();
        log(CKV_SIM_EV_TICK, (int)(alive[kInteractive].size() + alive[kMixed].size()), (int)alive[kBatch].size());
        dispatch();
    }
};

bool config_ok(const ckv_sim_config *c)
{
    return c && c->slots_interactive >= 1 && c->slots_batch >= 1 && c->rate_interactive > 0.0 && c->rate_batch > 0.0 &&
           c->startup_s >= 0.0 && c->tick_s > 0.0 && c->theta > 0.0 && c->theta <= 1.0 && c->delta >= 0.0 &&
           c->floor_instances >= 0 && c->initial_instances >= 0 && c->max_batch_instances >= 0 && c->groups_k >= 1 &&
           c->mu_o_prior >= 0.0 && c->sigma_o_prior >= 0.0 &&
           (c->policy == CKV_SIM_POLICY_CHIRON || c->policy == CKV_SIM_POLICY_IMMEDIATE);
}

}  // namespace

extern "C" int32_t global_autoscaler_simulate(const ckv_sim_config *cfg, int32_t n, const double *arrival_s,
                                              const int32_t *kind, const double *output_tokens, const double *ttft_slo_s,
                                              double *out_first_start_s, double *out_finish_s, int32_t *out_evictions,
                                              ckv_sim_summary *out_summary, double *log_time, int32_t *log_rows,
                                              int32_t log_cap, int64_t *out_log_rows)
{
    if (!config_ok(cfg) || n < 0 || (n > 0 && (!arrival_s || !kind || !output_tokens || !ttft_slo_s))) return kInval;
    if (log_cap < 0 || (log_cap > 0 && (!log_time || !log_rows))) return kInval;
    for (int32_t i = 0; i < n; ++i) {
        if (!(arrival_s[i] >= 0.0) || (i > 0 && arrival_s[i] < arrival_s[i - 1])) return kInval;
        if ((kind[i] != 0 && kind[i] != 1) || !(output_tokens[i] >= 1.0) || !(ttft_slo_s[i] > 0.0)) return kInval;
    }
    try {
        Simulation sim(*cfg, n, arrival_s, kind, output_tokens, ttft_slo_s, log_time, log_rows, log_cap);
        sim.run();
        for (int32_t i = 0; i < n; ++i) {
            if (out_first_start_s) out_first_start_s[i] = sim.reqs[i].first_start;
            if (out_finish_s) out_finish_s[i] = sim.reqs[i].finished_at;
            if (out_evictions) out_evictions[i] = sim.reqs[i].evictions;
        }
        if (out_summary) sim.summary(out_summary);
        if (out_log_rows) *out_log_rows = sim.events;
    } catch (const std::bad_alloc &) {
        return kNoMem;
    }
    return kOk;
}
