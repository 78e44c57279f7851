// Future-conditional overlap scheduling (Sec. 3.4 "Stream Throughput: Asynchronous Pipeline", Algorithm 1, Eq. 3): the
// control loop pops one action of the current chunk per control period and launches the inference of the next chunk
// K = ceil(mean inference latency / control period) actions before the chunk ends, conditioned on the state the robot
// will be in (approximated by the last commanded action). Host logic only: a small state machine that a control loop
// drives, and a discrete-event simulation of the loop over a trace of inference latencies (stall rate, staleness).
//
// Readings of the paper where it is silent: the mean latency is the arithmetic mean of the last 8 measurements (the
// initial estimate until the first one arrives); K is clamped to [0, C - 1], so the launch happens after action
// C - K, at the latest right after the first action of the chunk; a chunk that is not ready when the previous one
// ends stalls the loop (the last action is held) until it arrives.
#include <math.h>
#include <stdint.h>

#include <new>

#include "reflex.h"
#include "reflex_internal.cuh"

namespace {

constexpr int kWindow = 8;

int lookahead(double mean_inf, double tau_step, int C)
{
    int K = (int)ceil(mean_inf / tau_step - 1e-12);
    if (K < 0) K = 0;
    if (K > C - 1) K = C - 1;
    return K;
}

}  // namespace

struct reflex_overlap {
    int C;
    double tau_step;
    double lat[kWindow];
    int n_lat;            // measurements seen so far
    double init_inf;
    int chunk;            // index of the chunk being executed
    int i;                // actions of it executed so far (0..C)
    int K;                // lookahead fixed at the start of the chunk (Algorithm 1, line 3)
    int launched;         // the next chunk's inference has been requested
    int ready;            // ... and has been reported complete
    int64_t stalls;       // control periods spent waiting for a chunk
    double mean() const
    {
        if (n_lat == 0) return init_inf;
        const int n = n_lat < kWindow ? n_lat : kWindow;
        double s = 0.0;
        for (int j = 0; j < n; ++j) s += lat[j];
        return s / n;
    }
};

extern "C" {

int reflex_overlap_create(int C, double tau_step_s, double tau_inf_init_s, reflex_overlap_t **out)
{
    if (!out) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "out is NULL");
    if (C < 1 || !(tau_step_s > 0.0) || !(tau_inf_init_s >= 0.0)) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "C >= 1, tau_step > 0, tau_inf >= 0 required");
    reflex_overlap *s = new (std::nothrow) reflex_overlap();
    if (!s) return reflex::api_fail(REFLEX_ERR_CUDA, "out of host memory");
    s->C = C; s->tau_step = tau_step_s; s->n_lat = 0; s->init_inf = tau_inf_init_s;
    s->chunk = 0; s->i = 0; s->launched = 0; s->ready = 0; s->stalls = 0;
    s->K = lookahead(s->mean(), tau_step_s, C);
    *out = s;
    return REFLEX_OK;
}

int reflex_overlap_destroy(reflex_overlap_t *s)
{
    delete s;
    return REFLEX_OK;
}

int reflex_overlap_tick(reflex_overlap_t *s, reflex_overlap_event *ev)
{
    if (!s || !ev) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    ev->launch_now = 0; ev->stalled = 0; ev->lookahead = s->K;
    if (s->i == s->C) {
        // the chunk is used up: take the next one if it has arrived (Algorithm 1, line 11), else hold the last action
        if (!s->ready) {
            ++s->stalls;
            ev->stalled = 1; ev->chunk = s->chunk; ev->action = s->C - 1; ev->stalls_total = s->stalls;
            if (!s->launched) { s->launched = 1; ev->launch_now = 1; }   // (cannot happen with K <= C - 1; kept as a safeguard)
            return REFLEX_OK;
        }
        ++s->chunk; s->i = 0; s->launched = 0; s->ready = 0;
        s->K = lookahead(s->mean(), s->tau_step, s->C);                  // line 3
        ev->lookahead = s->K;
    }
    ev->chunk = s->chunk; ev->action = s->i;                             // line 5: execute queue.pop()
    ++s->i;
    if (!s->launched && s->i >= s->C - s->K) {                           // line 6: i = C - K (i counts from 1 there)
        s->launched = 1;
        ev->launch_now = 1;                                              // lines 7-8: condition on the action just commanded (Eq. 3)
    }
    ev->stalls_total = s->stalls;
    return REFLEX_OK;
}

int reflex_overlap_inference_done(reflex_overlap_t *s, double latency_s)
{
    if (!s) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (!s->launched || s->ready) return reflex::api_fail(REFLEX_ERR_STATE, "no inference in flight");
    if (!(latency_s >= 0.0)) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "latency must be >= 0");
    s->lat[s->n_lat % kWindow] = latency_s;
    ++s->n_lat;
    s->ready = 1;
    return REFLEX_OK;
}

int reflex_overlap_simulate(int C, double tau_step_s, double tau_inf_init_s, const double *tau_inf_s, int n_chunks, int mode, int fixed_K,
                            reflex_overlap_stats *out)
{
    if (!tau_inf_s || !out) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (C < 1 || n_chunks < 1 || !(tau_step_s > 0.0) || mode < 0 || mode > 2) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "bad argument");
    // Time is continuous; action j of a chunk that starts at t0 is executed at t0 + j tau_step. The inference of the next
    // chunk is launched right after action C - K (at t0 + (C - K) tau_step), takes tau_inf[c] and must be there at
    // t0 + C tau_step. mode 0: adaptive K (Algorithm 1); 1: synchronous (launch when the chunk has ended, K = 0 and no
    // overlap); 2: fixed K.
    double lat[kWindow];
    int n_lat = 0;
    double t0 = 0.0, stall_total = 0.0, stale_total = 0.0;
    int64_t stall_ticks = 0, k_sum = 0;
    int k_min = C, k_max = 0;
    for (int c = 0; c < n_chunks; ++c) {
        double mean = tau_inf_init_s;
        if (n_lat > 0) {
            const int n = n_lat < kWindow ? n_lat : kWindow;
            mean = 0.0;
            for (int j = 0; j < n; ++j) mean += lat[j];
            mean /= n;
        }
        int K = mode == 0 ? lookahead(mean, tau_step_s, C) : mode == 1 ? 0 : fixed_K;
        if (K < 0) K = 0;
        if (K > C - 1) K = C - 1;
        const double t_end = t0 + C * tau_step_s;
        const double t_launch = mode == 1 ? t_end : t0 + (C - K) * tau_step_s;
        if (!(tau_inf_s[c] >= 0.0)) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "latency %d is negative or NaN", c);
        const double t_ready = t_launch + tau_inf_s[c];
        const double stall = t_ready > t_end ? t_ready - t_end : 0.0;
        stall_total += stall;
        stall_ticks += (int64_t)ceil(stall / tau_step_s - 1e-9);
        stale_total += (t_end + stall) - t_launch;     // age of the conditioning state when the chunk's first action runs
        k_sum += K; if (K < k_min) k_min = K; if (K > k_max) k_max = K;
        lat[n_lat % kWindow] = tau_inf_s[c];
        ++n_lat;
        t0 = t_end + stall;
    }
    out->chunks = n_chunks;
    out->stall_ticks = stall_ticks;
    out->stall_time_s = stall_total;
    out->total_time_s = t0;
    out->mean_staleness_s = stale_total / n_chunks;
    out->mean_lookahead = (double)k_sum / n_chunks;
    out->min_lookahead = k_min;
    out->max_lookahead = k_max;
    return REFLEX_OK;
}

}  // extern "C"
