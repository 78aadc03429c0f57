// Repeat-offender bookkeeping of the node triage workflow (paper Section 6): a node that enters
// triage `limit` times within `period` seconds is marked for termination instead of going through
// triage again.  Host code only; per node a ring of its last `limit` entry times.
#include <cstdint>
#include <new>
#include <vector>

#include "../../include/guard_b200.h"
#include "kernels.h"

struct guard_triage {
    int nodes, limit;
    int64_t period;
    std::vector<int64_t> times;   // [nodes][limit] entry times, a ring per node
    std::vector<int32_t> count;   // [nodes] entries recorded so far (saturating)
    std::vector<int32_t> head;    // [nodes] ring position of the next entry
};

extern "C" {

int guard_triage_create(guard_triage **out, int nodes, int limit, int64_t period_s) {
    if (!out) return GUARD_ERR_ARG;
    *out = nullptr;
    if (nodes < 1 || limit < 1 || limit > 1024 || period_s < 0) {
        guard::set_global_error("guard_triage_create: need nodes >= 1, 1 <= limit <= 1024, period_s >= 0");
        return GUARD_ERR_ARG;
    }
    guard_triage *t = new (std::nothrow) guard_triage();
    if (!t) return GUARD_ERR_ARG;
    t->nodes = nodes;
    t->limit = limit;
    t->period = period_s;
    try {
        t->times.assign((size_t)nodes * limit, 0);
        t->count.assign((size_t)nodes, 0);
        t->head.assign((size_t)nodes, 0);
    } catch (...) {
        delete t;
        guard::set_global_error("guard_triage_create: out of host memory");
        return GUARD_ERR_ARG;
    }
    *out = t;
    return GUARD_OK;
}

int guard_triage_record(guard_triage *t, int node, int64_t time_s, int *entries_in_period) {
    if (!t || node < 0 || node >= t->nodes) return GUARD_ERR_ARG;
    int64_t *ring = t->times.data() + (size_t)node * t->limit;
    const int have = t->count[node];
    const int head = t->head[node];
    if (have > 0 && time_s < ring[(head + t->limit - 1) % t->limit]) return GUARD_ERR_ARG;   // time ran backwards
    ring[head] = time_s;
    t->head[node] = (head + 1) % t->limit;
    if (have < t->limit) t->count[node] = have + 1;
    // entries of the ring (at most `limit`, the newest included) no more than one period old
    int within = 0;
    for (int i = 0; i < t->count[node]; ++i) within += (time_s - ring[i] <= t->period);
    if (entries_in_period) *entries_in_period = within;
    return within >= t->limit ? 1 : 0;
}

void guard_triage_destroy(guard_triage *t) { delete t; }

}  // extern "C"
