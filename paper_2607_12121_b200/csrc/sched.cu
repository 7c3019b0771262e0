// Host-side policies of the paper's scheduler: the batch former (Sec. 4.3: patch monotasks, least-maximum-load
// packing) and the adaptive patch-granularity search (Sec. 4.1).  No device code.
#include <cmath>
#include <cstdint>

#include "../../include/flashdiff.h"

extern "C" {

fd_status fd_sched_pack(int n_devices, double* load, int n_tasks, const double* cost, const int32_t* home,
                        int32_t* assign_out) {
    if (n_devices < 1 || n_tasks < 0 || !load) return FD_ERR_INVALID_ARG;
    if (n_tasks > 0 && (!cost || !home || !assign_out)) return FD_ERR_INVALID_ARG;
    for (int g = 0; g < n_devices; ++g)
        if (!(load[g] >= 0.0) || !std::isfinite(load[g])) return FD_ERR_INVALID_ARG;
    for (int j = 0; j < n_tasks; ++j)
        if (!(cost[j] >= 0.0) || !std::isfinite(cost[j]) || home[j] >= n_devices) return FD_ERR_INVALID_ARG;

    for (int j = 0; j < n_tasks; ++j) {
        const double w = cost[j];
        // The straggler if j goes to g is max(largest load among the others, load[g] + w).  The largest and the
        // second largest load (with the position of the largest) give "largest among the others" for every g.
        int top = 0;
        double first = load[0], second = -1.0;
        for (int g = 1; g < n_devices; ++g) {
            if (load[g] > first) { second = first; first = load[g]; top = g; }
            else if (load[g] > second) second = load[g];
        }
        int best = -1;
        double best_worst = 0.0;
        bool home_ties = false;
        for (int g = 0; g < n_devices; ++g) {
            const double others = g == top ? second : first;
            const double mine = load[g] + w;
            const double worst = mine > others ? mine : others;
            if (best < 0 || worst < best_worst) {
                best = g; best_worst = worst; home_ties = g == home[j];
            } else if (worst == best_worst) {
                if (g == home[j]) home_ties = true;
                if (load[g] < load[best]) best = g;          // equal loads keep the smaller index
            }
        }
        const int g_star = home_ties ? home[j] : best;
        assign_out[j] = g_star;
        load[g_star] += w;
    }
    return FD_OK;
}

fd_status fd_sched_form_batch(int n, const int32_t* priority, const int64_t* arrival, const int32_t* active_tokens,
                              uint8_t* resident, int64_t token_budget, int max_resident, uint8_t* chosen_out) {
    if (n < 0 || token_budget < 0 || max_resident < 0) return FD_ERR_INVALID_ARG;
    if (n == 0) return FD_OK;
    if (!priority || !arrival || !active_tokens || !resident || !chosen_out) return FD_ERR_INVALID_ARG;
    int slots = max_resident;
    for (int i = 0; i < n; ++i) {
        if (active_tokens[i] < 0) return FD_ERR_INVALID_ARG;
        if (resident[i]) --slots;
    }
    // chosen_out doubles as the visit mark while the queue is drained: 2 = not visited yet
    for (int i = 0; i < n; ++i) chosen_out[i] = 2;
    int64_t left = token_budget;
    for (int k = 0; k < n; ++k) {
        int i = -1;                                            // head of the queue among the unvisited requests
        for (int c = 0; c < n; ++c) {
            if (chosen_out[c] != 2) continue;
            if (i < 0 || priority[c] > priority[i] || (priority[c] == priority[i] && arrival[c] < arrival[i])) i = c;
        }
        const int64_t t = active_tokens[i];
        bool take = t <= left;
        if (take && !resident[i]) {
            take = t > 0 && slots > 0;
            if (take) { resident[i] = 1; --slots; }
        }
        chosen_out[i] = take ? 1 : 0;
        if (take) left -= t;
    }
    return FD_OK;
}

// ---- adaptive patch granularity (Sec. 4.1) ----------------------------------------------------

static void rsearch_fail(fd_rsearch* st) {
    if (st->step == 1 && ++st->fails_at_one >= 2) st->converged = 1;
    st->dir = -st->dir;
    st->step = st->step / 2 > 1 ? st->step / 2 : 1;
}

fd_status fd_rsearch_init(fd_rsearch* st, int r_min, int r_max, int r_start) {
    if (!st || r_min < 1 || r_min > r_max || r_start < r_min || r_start > r_max) return FD_ERR_INVALID_ARG;
    st->r_min = r_min;
    st->r_max = r_max;
    st->accepted = st->candidate = r_start;
    const int half = (r_max - r_min + 1) / 2;
    st->step = half > 1 ? half : 1;
    st->dir = 1;
    st->have_ref = 0;
    st->fails_at_one = 0;
    st->converged = r_min == r_max;
    st->ref_perf = 0.0;
    return FD_OK;
}

fd_status fd_rsearch_update(fd_rsearch* st, double observed_perf, int32_t* next_r) {
    if (!st || !next_r || observed_perf != observed_perf) return FD_ERR_INVALID_ARG;
    if (!st->converged) {
        if (!st->have_ref) {
            st->have_ref = 1;
            st->ref_perf = observed_perf;
        } else if (observed_perf > st->ref_perf) {
            st->accepted = st->candidate;
            st->ref_perf = observed_perf;
            st->fails_at_one = 0;
        } else {
            rsearch_fail(st);
        }
        // next candidate; one that is clamped onto the accepted R is a failure that costs no run
        while (!st->converged) {
            int64_t c = (int64_t)st->accepted + (int64_t)st->dir * st->step;
            if (c < st->r_min) c = st->r_min;
            if (c > st->r_max) c = st->r_max;
            if ((int32_t)c != st->accepted) { st->candidate = (int32_t)c; break; }
            rsearch_fail(st);
        }
    }
    if (st->converged) st->candidate = st->accepted;
    *next_r = st->candidate;
    return FD_OK;
}

}  // extern "C"
