// C ABI of the library: context object, workspace carving, argument checks and the
// stream-ordered kernel sequences behind guard_ingest / guard_score / guard_sweep_qualify.
#include <atomic>
#include <chrono>
#include <cstdarg>
#include <cstddef>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/guard_b200.h"
#include "kernels.h"

using namespace guard;

namespace {

constexpr size_t kAlign = 256;
#ifndef GUARD_EVAL_PRIO
#define GUARD_EVAL_PRIO 1
#endif
#ifndef GUARD_INGEST_STREAMS
#define GUARD_INGEST_STREAMS 2
#endif
constexpr int kIngestStreams = GUARD_INGEST_STREAMS;   // internal streams the cross-rank kernels of consecutive blocks take turns on (deferred mode)
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
    size_t status, consec, lastflag, lasttier, topk_idx, topk_hint, ticket, fleet, xr_small, xr_grid, inc_rbc, wmed, wmed_stride, stepstat, topk_cand, wspread, wcentre, kcnt, inc_lo, inc_hi, inc_cnt, inc_val, inc_rbl, xr_big, xr_big_stride, mask, ring, total;
    int xr_steps;   // steps per launch of the multi-kernel bracketed cross-rank path (0: not used)
    int xr_cluster; // the cluster-per-step cross-rank path applies
    int xr_split;   // the six-kernel split cross-rank path applies
    int xr_gridp;   // single rows keep brackets between calls (two ColHintState at xr_grid: ingest, fleet baseline)
};

// State and scratch first, the two rings last (the telemetry ring is by far the largest).
Layout make_layout(int R, int M, int C, int K) {
    Layout L{};
    size_t off = 0;
    L.status = off;    off = align_up(off + 64);
    L.ticket = off;    off = align_up(off + 64);
    L.fleet = off;     off = align_up(off + 3 * kMaxMetrics * sizeof(float));
    L.consec = off;    off = align_up(off + (size_t)R);
    L.lastflag = off;  off = align_up(off + (size_t)R);
    L.lasttier = off;  off = align_up(off + (size_t)R);
    L.topk_idx = off;  off = align_up(off + 2 * align_up((size_t)(K > 0 ? K : 1) * sizeof(int32_t)));
    L.topk_hint = off; off = align_up(off + 256 + 1024 * sizeof(unsigned long long));   // TopkHint, then the hinted pass's list
    L.xr_split = xrank_split_supported(R, M) ? 1 : 0;
    L.xr_cluster = (!L.xr_split && xrank_cluster_supported(R, M)) ? 1 : 0;
    L.xr_steps = (!L.xr_split && !L.xr_cluster && xrank_bracket_supported(R, M)) ? xrank_scratch_steps(R, M, C) : 0;
    L.xr_small = off;  off = align_up(off + (L.xr_steps ? xrank_scratch_small_bytes(M, L.xr_steps) : 0));
    L.xr_gridp = (xrank_column_supported(R) && R >= 8192) ? 1 : 0;
    L.xr_grid = off;   off = align_up(off + 2 * align_up(sizeof(ColHintState)));
    L.inc_rbc = off;   off = align_up(off + 64);   // rebuild list counter and ticket (zero before first use)
    // the windowed medians and the kept top-k indices exist twice: consecutive evaluations alternate, so that a
    // deferred evaluation's tail may still read its medians while the next evaluation's window kernels write theirs
    L.wmed = off;      off = align_up(off + (size_t)R * M * sizeof(float));
    L.wmed_stride = off - L.wmed;
    off = align_up(off + (size_t)R * M * sizeof(float));
    L.stepstat = off;  off = align_up(off + 2 * (size_t)C * M * sizeof(float));
    L.topk_cand = off; off = align_up(off + (size_t)topk_blocks(R) * (K > 0 ? K : 1) * sizeof(unsigned long long));
    L.wspread = off;   off = align_up(off + (size_t)R * M * sizeof(float));
    L.wcentre = off;   off = align_up(off + (size_t)R * M * sizeof(float));
    L.kcnt = off;      off = align_up(off + (size_t)R * M * sizeof(uint16_t));   // k-of-W counts of the last evaluation's window
    // sliding-window state: interval ends, packed counts, listed values
    L.inc_lo = off;    off = align_up(off + window_inc_bytes(R * M));
    L.inc_hi = off;    off = align_up(off + window_inc_bytes(R * M));
    L.inc_cnt = off;   off = align_up(off + window_inc_bytes(R * M));
    L.inc_val = off;   off = align_up(off + (size_t)kIncSlots * window_inc_bytes(R * M));
    L.inc_rbl = off;   off = align_up(off + window_inc_bytes(R * M));   // series a sliding launch has to rebuild
    L.xr_big = off;    off = align_up(off + (L.xr_split ? xrank_split_scratch_bytes(R, M, C < kSplitMaxSteps ? C : kSplitMaxSteps)
                                             : L.xr_steps ? xrank_scratch_big_bytes(R, M, L.xr_steps) : 0));
    // in deferred mode consecutive blocks run their cross-rank kernels on streams of their own
    L.xr_big_stride = off - L.xr_big;   // further copies of the split scratch, one per internal ingest stream
    off = align_up(off + (L.xr_split ? (kIngestStreams - 1) * L.xr_big_stride : 0));
    L.mask = off;      off = align_up(off + (size_t)C * R * (M <= 8 ? 1 : 4));
    L.ring = off;      off = align_up(off + (size_t)C * R * M * sizeof(float));
    L.total = off;
    return L;
}

bool sizes_ok(int R, int M, int W, int C, int K) {
    return R >= 1 && M >= 1 && M <= GUARD_MAX_METRICS && W >= 1 && W <= GUARD_MAX_WINDOW && C >= W && K >= 0 &&
           K <= GUARD_MAX_TOPK && K <= R && (long long)R * M <= 0x7FFFFFFFLL;
}

thread_local char g_error[256] = "";

void set_error(char *dst, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(dst, 256, fmt, ap);
    va_end(ap);
}

// Copies and checks the per-metric parameters; returns nullptr or an error text.
const char *fill_params(MetricParams &p, const guard_thresholds *th, int M, int k, bool online) {
    if (!th || !th->dir || !th->thr || !th->floor_rel || !th->floor_abs) return "thresholds or one of its arrays is NULL";
    memset(&p, 0, sizeof(p));
    p.M = M;
    p.k = k;
    p.primary = th->primary;
    p.min_signals = th->min_signals;
    p.n_consec = th->n_consec;
    p.tier_moderate = th->tier_moderate;
    p.tier_severe = th->tier_severe;
    if (online) {
        if (th->primary < 0 || th->primary >= M) return "primary metric index out of range";
        if (th->min_signals < 1) return "min_signals must be >= 1";
        if (th->n_consec < 1 || th->n_consec > 255) return "n_consec must be in 1..255";
        if (!(th->tier_moderate >= 0.0f) || !(th->tier_severe >= th->tier_moderate)) return "tier thresholds must satisfy 0 <= moderate <= severe";
        if (th->ranks_per_node < 1) return "ranks_per_node must be >= 1";
    }
    for (int m = 0; m < M; ++m) {
        if (th->dir[m] != 1 && th->dir[m] != -1) return "dir[m] must be +1 or -1";
        if (!(th->thr[m] >= 0.0f) || !(th->thr[m] < 1e30f)) return "thr[m] must be finite and >= 0";
        if (!(th->floor_rel[m] >= 0.0f) || !(th->floor_abs[m] >= 0.0f)) return "floors must be >= 0";
        p.dir[m] = th->dir[m];
        p.thrp[m] = (float)((double)th->thr[m] / 0.6745);
        p.floor_rel[m] = th->floor_rel[m];
        p.floor_abs[m] = th->floor_abs[m];
    }
    return nullptr;
}

}  // namespace

namespace guard {
void set_global_error(const char *text) { set_error(g_error, "%s", text); }
}  // namespace guard

namespace {

int status_to_code(uint32_t s) {
    if (s & kStatNonFinite) return GUARD_ERR_NONFINITE;
    if (s & kStatTimeout) return GUARD_ERR_TIMEOUT;
    if (s & kStatInternal) return GUARD_ERR_INTERNAL;
    return GUARD_OK;
}

}  // namespace

struct guard_ctx {
    int R, M, W, k, C, K;
    MetricParams p;
    Layout L;
    char *ws;
    long long seen;
    long long launches;  // kernels enqueued by this context so far
    long long evals;     // evaluations since creation / reset
    long long seen_at_eval = 0;   // steps seen at the last evaluation
    int ranks_per_node = 8;
    long long wait_limit = 0;     // test hook: limit of the warp window path's first wait (0: default)
    // Sliding-window state (window.cu): current for the window of inc_n steps ending at step count inc_seen
    // (-1: none).  hints_ready: a whole-window kernel has seeded the per-series search intervals.
    long long inc_seen = -1;
    int inc_n = 0;
    long long cnt_seen = -1;      // the k-of-W counts kept in the workspace hold for the window of cnt_n steps ending here
    int cnt_n = 0;
    bool sliding = true;          // guard_set_sliding
    bool hints_ready = false;
    // overlap of the window medians (which need only the ring) with the cross-rank kernels of the
    // ingest that precedes them: an internal stream forked from and joined into the caller's
    bool overlap = true;
    bool fork_fresh = false;          // ev_fork was recorded by an ingest not yet followed by an evaluation
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_topk = nullptr;
    bool ensure_side() {
        if (side) return true;
        // the evaluation's streams get the highest priority: flags should not queue behind the next blocks' sweeps
        int prio_lo = 0, prio_hi = 0;
        cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
        if (cudaStreamCreateWithPriority(&side, cudaStreamNonBlocking, GUARD_EVAL_PRIO ? prio_hi : 0) != cudaSuccess) { side = nullptr; return false; }
        if (cudaEventCreateWithFlags(&ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ev_join, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ev_topk, cudaEventDisableTiming) != cudaSuccess) {
            cudaStreamDestroy(side);
            side = nullptr;
            return false;
        }
        return true;
    }
    // Deferred evaluations: guard_score enqueues the evaluation on internal streams and does not
    // make the caller's stream wait for it, so that the evaluation's short, latency-bound tail runs
    // beside the next guard_ingest.  At most one evaluation is pending; the next guard_score,
    // guard_join, guard_sync_status, guard_reset and guard_destroy wait for it.
    bool deferred = false;
    bool pending = false;             // an evaluation has been enqueued whose end the caller's stream has not waited for
    int pending_n = 0;                // its window length
    long long pending_seen = 0;       // steps seen when it was enqueued (its window ends there)
    // In deferred mode the cross-rank kernels of consecutive ingests alternate between two internal
    // streams (each with its own scratch), so that one block's selections overlap the next block's
    // sweeps; the caller's stream waits for them only where it joins.
    cudaStream_t xs[kIngestStreams] = {};
    cudaEvent_t ev_xs[kIngestStreams] = {}, ev_data = nullptr;
    bool xs_busy[kIngestStreams] = {};   // stream k has work the caller's stream has not waited for
    long long xs_first[kIngestStreams] = {};   // first step (counted from creation / reset) of the oldest such block
    int xs_next = 0;
    int scratch_sel = 0;                // which split scratch the next launch uses
    cudaStream_t tail = nullptr;
    cudaStream_t aux = nullptr;       // deferred evaluations: the top-k selection, beside the fleet baseline and clear of the window medians' stream
    cudaEvent_t ev_x = nullptr, ev_w = nullptr;
    // end of the deferred evaluations, by parity of the evaluation count: up to two may be in flight (the tail of
    // one beside the window medians of the next); each keeps its window for the ring protection
    cudaEvent_t ev_e[2] = {nullptr, nullptr};
    struct Inflight { bool on = false; long long seen = 0; int n = 0; } infl[2];
    int last_q = 0;                   // parity of the pending evaluation
    bool ensure_xs() {
        if (xs[0]) return true;
        if (!ensure_tail()) return false;
        bool ok = cudaEventCreateWithFlags(&ev_data, cudaEventDisableTiming) == cudaSuccess;
        for (int k = 0; k < kIngestStreams && ok; ++k)
            ok = cudaStreamCreateWithFlags(&xs[k], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&ev_xs[k], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            for (int k = 0; k < kIngestStreams; ++k) {
                if (xs[k]) cudaStreamDestroy(xs[k]);
                if (ev_xs[k]) cudaEventDestroy(ev_xs[k]);
                xs[k] = nullptr;
                ev_xs[k] = nullptr;
            }
            if (ev_data) cudaEventDestroy(ev_data);
            ev_data = nullptr;
        }
        return ok;
    }
    // Ring slots (in steps, counted back from the newest) that work not yet joined still reads.
    // Oldest step that work not yet joined may still read: a pending evaluation reads the pending_n
    // steps that ended where `seen` stood when it was enqueued; an internal ingest stream reads the
    // blocks enqueued on it since it was last joined.  Everything from that step on is protected.
    // Work whose end event has already completed (a host-side query, no waiting) reads nothing any more.
    long long protected_steps(int need) {
        long long first = seen;
        for (int q = 0; q < 2; ++q)
            if (infl[q].on && infl[q].seen - infl[q].n < first) first = infl[q].seen - infl[q].n;
        for (int k = 0; k < kIngestStreams; ++k)
            if (xs_busy[k] && xs_first[k] < first) first = xs_first[k];
        if (need + (seen - first) <= C) return seen - first;   // no conflict even if all of it is still running: nothing to query
        first = seen;
        for (int q = 0; q < 2; ++q)
            if (infl[q].on) {
                if (cudaEventQuery(ev_e[q]) == cudaSuccess) { infl[q].on = false; continue; }   // finished: reads nothing any more
                if (infl[q].seen - infl[q].n < first) first = infl[q].seen - infl[q].n;
            }
        for (int k = 0; k < kIngestStreams; ++k)
            if (xs_busy[k] && xs_first[k] < first) {
                if (cudaEventQuery(ev_xs[k]) == cudaSuccess) { xs_busy[k] = false; continue; }   // finished: nothing left to wait for
                first = xs_first[k];
            }
        (void)cudaGetLastError();   // cudaErrorNotReady is an answer, not an error
        return seen - first;
    }
    bool ensure_tail() {
        if (tail) return true;
        if (!ensure_side()) return false;
        int prio_lo = 0, prio_hi = 0;
        cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
        if (cudaStreamCreateWithPriority(&tail, cudaStreamNonBlocking, GUARD_EVAL_PRIO ? prio_hi : 0) != cudaSuccess) { tail = nullptr; return false; }
        if (cudaStreamCreateWithPriority(&aux, cudaStreamNonBlocking, GUARD_EVAL_PRIO ? prio_hi : 0) != cudaSuccess) aux = nullptr;
        if (cudaEventCreateWithFlags(&ev_x, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ev_w, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ev_e[0], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ev_e[1], cudaEventDisableTiming) != cudaSuccess) {
            cudaStreamDestroy(tail);
            tail = nullptr;
            return false;
        }
        return true;
    }
    // Makes `st` wait for the pending evaluation, if any.
    cudaError_t join(cudaStream_t st) {
        cudaError_t e = cudaSuccess;
        if (pending) {   // the tail stream runs the evaluations in order: the latest one's end covers the one before
            e = cudaStreamWaitEvent(st, ev_e[last_q], 0);
            if (e == cudaSuccess) { pending = false; infl[0].on = false; infl[1].on = false; }
        }
        return e;
    }
    // Makes `st` wait for the cross-rank kernels still running on the internal ingest streams.
    cudaError_t join_xs(cudaStream_t st) {
        for (int k = 0; k < kIngestStreams; ++k)
            if (xs_busy[k]) {
                cudaError_t e = cudaStreamWaitEvent(st, ev_xs[k], 0);
                if (e != cudaSuccess) return e;
                xs_busy[k] = false;
            }
        return cudaSuccess;
    }
    int profiling = 0;                                        // 1: time the MAD sweep of every ingest, 2: the window kernel of every evaluation
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof;    // recorded, not yet read
    char error[256];

    uint32_t *status() const { return (uint32_t *)(ws + L.status); }
    unsigned int *ticket() const { return (unsigned int *)(ws + L.ticket); }
    float *fleet_med() const { return (float *)(ws + L.fleet); }
    float *fleet_mad() const { return fleet_med() + kMaxMetrics; }
    uint8_t *consec() const { return (uint8_t *)(ws + L.consec); }
    uint8_t *lastflag() const { return (uint8_t *)(ws + L.lastflag); }
    uint8_t *lasttier() const { return (uint8_t *)(ws + L.lasttier); }
    int32_t *topk_idx(int q) const { return (int32_t *)(ws + L.topk_idx + (size_t)q * align_up((size_t)(K > 0 ? K : 1) * sizeof(int32_t))); }
    float *wmed(int q) const { return (float *)(ws + L.wmed + (size_t)q * L.wmed_stride); }
    int eval_q() const { return (int)(evals & 1); }        // buffers of the evaluation about to be made
    int prev_q() const { return (int)((evals + 1) & 1); }  // ... and of the one made last
    float *step_med() const { return (float *)(ws + L.stepstat); }
    float *step_mad() const { return step_med() + (size_t)C * M; }
    unsigned long long *topk_cand() const { return (unsigned long long *)(ws + L.topk_cand); }
    void *mask() const { return ws + L.mask; }
    float *ring() const { return (float *)(ws + L.ring); }
    int mask_bytes() const { return M <= 8 ? 1 : 4; }
    // Cross-rank statistics of S rows: the bracketed path where it applies, else the direct one.
    // own_scratch = false: the call may run beside another cross-rank call of this context (the fleet
    // baseline of a deferred evaluation beside the next ingest), so it must not touch the one
    // scratch of the bracketed path: such rows take the direct selection.
    // site: 0 the ingested step, 1 the fleet baseline, -1 neither.  A site keeps the brackets of its single rows.
    bool row_hints = true;   // guard_set_row_hints
    // stamp of the split path's column records: changed whenever the scratch stops describing this context's data
    uint32_t split_epoch = 1;
    // never the same value twice in a process (device memory is handed out again with its old contents, at the
    // same addresses: a stamp derived from addresses would take another context's leftovers for its own)
    void new_epoch() {
        static std::atomic<uint32_t> next{(uint32_t)std::chrono::steady_clock::now().time_since_epoch().count() | 1u};
        do { split_epoch = next.fetch_add(1u); } while (split_epoch == 0u);
    }
    ColHintState *hint_state(int site) const { return (ColHintState *)(ws + L.xr_grid + (size_t)site * align_up(sizeof(ColHintState))); }
    cudaError_t xrank(XrankArgs a, int S, cudaStream_t st, bool own_scratch = true, int site = -1) {
        // a few rows at a time: one CTA per column keeps the whole GPU busy
        if (xrank_column_supported(R) && (long long)S * M <= 64 && !a.cut) {
            // one row of a wide fleet: bracketed by the call site's previous result
            if (S == 1 && site >= 0 && L.xr_gridp && row_hints) a.hint = hint_state(site);
            launches += 1;
            return launch_xrank_column(a, p, S, st);
        }
        if (L.xr_split && a.mask_bytes == 1) {
            a.fallbacks = status() + 1;
            a.hint_epoch = row_hints ? split_epoch : 0u;
            const int first = a.first_slot;
            const int smax = C < kSplitMaxSteps ? C : kSplitMaxSteps;
            for (int s0 = 0; s0 < S; s0 += smax) {
                const int n = (S - s0 < smax) ? (S - s0) : smax;
                XrankArgs g = a;
                g.first_slot = (int)(((long long)first + s0) % a.capacity);
                g.med = a.med + (size_t)s0 * M;
                g.mad = a.mad + (size_t)s0 * M;
                if (a.med_user) g.med_user = a.med_user + (size_t)s0 * M;
                if (a.mad_user) g.mad_user = a.mad_user + (size_t)s0 * M;
                cudaError_t e = launch_xrank_split(g, p, n, ws + L.xr_big + (size_t)scratch_sel * L.xr_big_stride, status() + 2, st,
                                                   (profiling == 1 && a.mask_base) ? &prof : nullptr);
                if (e != cudaSuccess) return e;
                launches += 6;
            }
            return cudaSuccess;
        }
        if (L.xr_cluster && a.mask_bytes == 1) {
            a.fallbacks = status() + 1;
            launches += 1;
            return launch_xrank_cluster(a, p, S, status() + 2, st, (profiling == 1 && a.mask_base) ? &prof : nullptr);
        }
        if (L.xr_steps == 0 || !own_scratch) { launches += 1; return launch_xrank_direct(a, p, S, st); }
        XrankScratch sc = carve_xrank_scratch(ws + L.xr_small, ws + L.xr_big, R, M, L.xr_steps);
        sc.reasons = status() + 2;
        const int first = a.first_slot;
        for (int s0 = 0; s0 < S; s0 += L.xr_steps) {
            const int n = (S - s0 < L.xr_steps) ? (S - s0) : L.xr_steps;
            XrankArgs g = a;
            g.fallbacks = status() + 1;
            g.first_slot = (int)(((long long)first + s0) % a.capacity);
            g.med = a.med + (size_t)s0 * M;
            g.mad = a.mad + (size_t)s0 * M;
            if (a.med_user) g.med_user = a.med_user + (size_t)s0 * M;
            if (a.mad_user) g.mad_user = a.mad_user + (size_t)s0 * M;
            cudaError_t e = launch_xrank_bracketed(g, p, sc, n, st);
            if (e != cudaSuccess) return e;
            launches += 6;
        }
        return cudaSuccess;
    }
    // The window kernel, with a pair of events around it on its stream while profiling mode 2 is on.
    const IncArgs *inc_now = nullptr;   // set by guard_score while its window medians take the sliding update
    cudaError_t window(const WindowArgs &w, cudaStream_t ws_) {
        auto go = [&]() { return inc_now ? launch_window_incremental(w, *inc_now, ws_) : launch_window_select(w, ws_); };
        if (profiling != 2) return go();
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return cudaGetLastError();
        cudaEventRecord(e0, ws_);
        const cudaError_t e = go();
        cudaEventRecord(e1, ws_);
        prof.emplace_back(e0, e1);
        return e;
    }
    int fail(int code, const char *fmt, ...) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(error, sizeof(error), fmt, ap);
        va_end(ap);
        return code;
    }
    int cuda_fail(cudaError_t e, const char *what) { return fail(GUARD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e)); }
};

extern "C" {

size_t guard_workspace_bytes(int ranks, int metrics, int W, int capacity_steps, int topk) {
    if (!sizes_ok(ranks, metrics, W, capacity_steps, topk)) return 0;
    return make_layout(ranks, metrics, capacity_steps, topk).total;
}

int guard_create(guard_ctx **out, int ranks, int metrics, int W, int k, const guard_thresholds *th, int capacity_steps,
                 int topk, void *d_workspace, size_t workspace_bytes, void *stream) {
    if (!out) { set_error(g_error, "out is NULL"); return GUARD_ERR_ARG; }
    *out = nullptr;
    if (!sizes_ok(ranks, metrics, W, capacity_steps, topk)) {
        set_error(g_error, "invalid sizes: need ranks >= 1, 1 <= metrics <= %d, 1 <= W <= %d, capacity >= W, 0 <= topk <= min(ranks, %d)",
                  GUARD_MAX_METRICS, GUARD_MAX_WINDOW, GUARD_MAX_TOPK);
        return GUARD_ERR_ARG;
    }
    if (k < 1 || k > W) { set_error(g_error, "k must be in 1..W"); return GUARD_ERR_ARG; }
    MetricParams p;
    if (const char *msg = fill_params(p, th, metrics, k, true)) { set_error(g_error, "%s", msg); return GUARD_ERR_ARG; }
    const Layout L = make_layout(ranks, metrics, capacity_steps, topk);
    if (!d_workspace || ((uintptr_t)d_workspace % kAlign) != 0 || workspace_bytes < L.total) {
        set_error(g_error, "workspace must be non-NULL, 256-byte aligned and at least %zu bytes", L.total);
        return GUARD_ERR_WORKSPACE;
    }
    guard_ctx *c = new (std::nothrow) guard_ctx();
    if (!c) { set_error(g_error, "out of host memory"); return GUARD_ERR_ARG; }
    c->R = ranks; c->M = metrics; c->W = W; c->k = k; c->C = capacity_steps; c->K = topk;
    c->p = p; c->L = L; c->ws = (char *)d_workspace; c->seen = 0; c->launches = 0; c->evals = 0; c->error[0] = 0;
    c->ranks_per_node = th->ranks_per_node;
    c->new_epoch();
    // state: status word, ticket, fleet statistics, consecutive counters
    cudaError_t e = cudaMemsetAsync(c->ws, 0, L.wmed, (cudaStream_t)stream);
    if (e != cudaSuccess) {
        set_error(g_error, "cudaMemsetAsync: %s", cudaGetErrorString(e));
        delete c;
        return GUARD_ERR_CUDA;
    }
    *out = c;
    return GUARD_OK;
}

int guard_ring_reserve(guard_ctx *c, int steps, float **d_slot) {
    if (!c) return GUARD_ERR_ARG;
    if (!d_slot || steps < 1 || steps > c->C) return c->fail(GUARD_ERR_ARG, "steps must be in 1..capacity and d_slot non-NULL");
    const int slot = (int)(c->seen % c->C);
    if (slot + steps > c->C) return c->fail(GUARD_ERR_ARG, "reserved span would wrap around the ring (slot %d + %d > %d)", slot, steps, c->C);
    if (steps + c->protected_steps(steps) > c->C)
        return c->fail(GUARD_ERR_NOT_READY, "the reserved slots are still read by deferred work: call guard_join first");
    *d_slot = c->ring() + (size_t)slot * c->R * c->M;
    return GUARD_OK;
}

int guard_ingest(guard_ctx *c, const float *d_block, int B, float *d_step_med, float *d_step_mad, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    if (!d_block) return c->fail(GUARD_ERR_ARG, "d_block is NULL");
    if (B < 1 || B > c->C) return c->fail(GUARD_ERR_ARG, "B must be in 1..capacity_steps (%d)", c->C);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t row = (size_t)c->R * c->M;
    const int slot = (int)(c->seen % c->C);
    const bool in_place = (d_block == c->ring() + (size_t)slot * row) && (slot + B <= c->C);
    if (B + c->protected_steps(B) > c->C) {   // this block's slots are still read by deferred work
        cudaError_t e = c->join(st);
        if (e == cudaSuccess) e = c->join_xs(st);
        if (e != cudaSuccess) return c->cuda_fail(e, "join of deferred work");
    }
    if (!in_place) {
        const int first = (slot + B <= c->C) ? B : (c->C - slot);
        cudaError_t e = cudaMemcpyAsync(c->ring() + (size_t)slot * row, d_block, (size_t)first * row * sizeof(float),
                                        cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && first < B)
            e = cudaMemcpyAsync(c->ring(), d_block + (size_t)first * row, (size_t)(B - first) * row * sizeof(float),
                                cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return c->cuda_fail(e, "cudaMemcpyAsync(ring)");
    }
    // the ring now holds the block (in stream order): evaluations may start reading it from here
    c->fork_fresh = false;
    if (c->overlap && c->ensure_side() && cudaEventRecord(c->ev_fork, st) == cudaSuccess) c->fork_fresh = true;
    XrankArgs a{};
    a.base = c->ring();
    a.row_stride = (long long)row;
    a.first_slot = slot;
    a.capacity = c->C;
    a.R = c->R;
    a.M = c->M;
    a.med = c->step_med();
    a.mad = c->step_mad();
    a.med_user = d_step_med;
    a.mad_user = d_step_mad;
    a.cut = nullptr;
    a.mask_base = c->mask();
    a.mask_bytes = c->mask_bytes();
    a.check_finite = 1;
    a.status = c->status();
    cudaError_t e;
    const bool piped = c->deferred && c->L.xr_split && a.mask_bytes == 1 && (long long)B * c->M > 64 && !d_step_med &&
                       !d_step_mad && c->ensure_xs();
    if (piped) {
        const int k = c->xs_next;
        c->xs_next = (k + 1) % kIngestStreams;
        e = cudaEventRecord(c->ev_data, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c->xs[k], c->ev_data, 0);
        if (e != cudaSuccess) return c->cuda_fail(e, "fork of the ingest stream");
        c->scratch_sel = k;
        e = c->xrank(a, B, c->xs[k]);
        c->scratch_sel = 0;
        if (e == cudaSuccess) e = cudaEventRecord(c->ev_xs[k], c->xs[k]);
        if (!c->xs_busy[k]) c->xs_first[k] = c->seen;
        c->xs_busy[k] = true;
    } else {
        e = c->join_xs(st);   // earlier blocks still on the internal streams come first
        if (e == cudaSuccess) e = c->xrank(a, B, st, true, 0);
    }
    if (e != cudaSuccess) return c->cuda_fail(e, "xrank launch");
    c->seen += B;
    return GUARD_OK;
}

int guard_score(guard_ctx *c, float *d_wmed, float *d_fleet_med, float *d_fleet_mad, float *d_scores, uint16_t *d_counts,
                uint32_t *d_metric_mask, uint8_t *d_flags, uint8_t *d_tier, int32_t *d_topk_idx, float *d_topk_score,
                void *stream) {
    if (!c) return GUARD_ERR_ARG;
    if (c->seen < 1) return c->fail(GUARD_ERR_NOT_READY, "guard_score before the first ingested step");
    cudaStream_t st = (cudaStream_t)stream;
    const int n = (int)(c->seen < c->W ? c->seen : c->W);
    const int last = (int)((c->seen - 1) % c->C);
    const size_t row = (size_t)c->R * c->M;

    WindowArgs w{};
    w.ring = c->ring();
    w.row_stride = (long long)row;
    w.capacity = c->C;
    w.last_slot = last;
    w.n = n;
    w.series = (int)row;
    const int q = c->eval_q();
    w.wmed = c->wmed(q);
    w.wmed_prev = c->wmed(q ^ 1);
    w.wmed_user = d_wmed;
    w.use_hint = c->hints_ready ? 1 : 0;
    w.spread = (float *)(c->ws + c->L.wspread);
    w.centre = (float *)(c->ws + c->L.wcentre);
    // windows that share at least three quarters of their steps with the previous evaluation's: the
    // previous median itself is the centre, and a much narrower interval does
    if (c->evals > 0 && (c->seen - c->seen_at_eval) * 4 <= n) { w.target = kWindowNearTarget; w.smooth = kWindowNearSmooth; }
    // Evaluations that follow one another by a few steps: the sliding update reads only the steps that
    // entered and left the window since its per-series state was current (or rebuilds that state).
    IncArgs ia{};
    const long long gap = c->evals > 0 ? c->seen - c->seen_at_eval : c->seen;   // steps since the previous evaluation
    // the steps that leave the window must still be in the ring when the next evaluation slides: a ring of
    // exactly W steps has overwritten them, and rebuilding every series every time would cost more than the
    // whole-window kernels
    const bool use_inc = c->sliding && gap <= kIncMaxNew && window_inc_supported(w) && (long long)c->C >= n + (gap > 0 ? gap : 1);
    if (use_inc) {
        ia.lo = (float *)(c->ws + c->L.inc_lo);
        ia.hi = (float *)(c->ws + c->L.inc_hi);
        ia.cnt = (uint32_t *)(c->ws + c->L.inc_cnt);
        ia.val = (float *)(c->ws + c->L.inc_val);
        ia.rebuilds = c->status() + 14;
        ia.rb_list = (uint32_t *)(c->ws + c->L.inc_rbl);
        ia.rb_count = (uint32_t *)(c->ws + c->L.inc_rbc);
        const long long p1 = c->inc_seen, p0 = p1 - c->inc_n, q1 = c->seen, q0 = q1 - n;
        // the windows overlap, few steps entered / left, and the steps that left are still in the ring
        if (p1 >= 0 && q0 < p1 && q1 - p1 <= kIncMaxNew && q0 - p0 <= kIncMaxNew && q1 - p0 <= c->C) {
            ia.entering = (int)(q1 - p1);
            ia.leaving = (int)(q0 - p0);
        } else {
            ia.rebuild_all = 1;
        }
        c->inc_seen = c->seen;
        c->inc_n = n;
    } else {
        c->hints_ready = true;   // a whole-window kernel runs: it seeds (or re-tunes) the per-series search intervals
    }
    c->inc_now = use_inc ? &ia : nullptr;
    c->seen_at_eval = c->seen;
    w.fb_count = c->status() + 8;
    w.fb_list = (uint32_t *)(c->ws + c->L.inc_rbl);          // shared with the sliding path's rebuild list: an evaluation takes one path
    w.fb_list_count = (uint32_t *)(c->ws + c->L.inc_rbc);
    w.status = c->status();
    w.first_wait_cycles = c->wait_limit;
    // The window medians read only the ring: run them on the internal stream, forked where the
    // ring became complete, so that they overlap the cross-rank kernels of the preceding ingest;
    // the caller's stream waits for them before anything that uses them.
    cudaError_t e;
    // a deferred evaluation still pending is complete, in the caller's stream order, from here on
    const bool same_buffers_busy = c->infl[q].on;   // the evaluation before the previous one (join clears the records)
    e = c->join(st);
    if (e != cudaSuccess) return c->cuda_fail(e, "join of the deferred evaluation");
    const bool forked = c->overlap && c->fork_fresh && c->side;
    c->fork_fresh = false;
    const bool defer = c->deferred && c->ensure_tail();
    if (!defer) {
        e = c->join_xs(st);
        if (e != cudaSuccess) return c->cuda_fail(e, "join of the ingest streams");
    }
    cudaStream_t ts = st;   // stream of the evaluation's tail: fleet baseline, scores / flags, top-k
    if (defer) {
        // window medians on the internal stream (after the ring is complete and after the previous
        // evaluation's tail, which still reads the medians they overwrite); the tail on a stream of
        // its own after them and after this block's cross-rank kernels; the caller's stream waits
        // for none of it
        if (!forked) {
            e = cudaEventRecord(c->ev_fork, st);
            if (e != cudaSuccess) return c->cuda_fail(e, "event record");
        }
        e = cudaStreamWaitEvent(c->side, c->ev_fork, 0);
        // the evaluation before the previous one used the same buffers: its tail must have read them
        if (e == cudaSuccess && same_buffers_busy) e = cudaStreamWaitEvent(c->side, c->ev_e[q], 0);
        if (e == cudaSuccess) e = c->window(w, c->side);
        if (e == cudaSuccess) e = cudaEventRecord(c->ev_w, c->side);
        if (e == cudaSuccess) e = cudaEventRecord(c->ev_x, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c->tail, c->ev_w, 0);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c->tail, c->ev_x, 0);
        for (int k = 0; k < kIngestStreams && e == cudaSuccess; ++k)   // cross-rank kernels of the window's blocks on the ingest streams
            if (c->xs_busy[k]) e = cudaStreamWaitEvent(c->tail, c->ev_xs[k], 0);
        ts = c->tail;
    } else if (forked) {
        e = cudaStreamWaitEvent(c->side, c->ev_fork, 0);
        if (e == cudaSuccess) e = c->window(w, c->side);
        if (e == cudaSuccess) e = cudaEventRecord(c->ev_join, c->side);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_join, 0);
    } else {
        e = c->window(w, st);
    }
    c->inc_now = nullptr;
    if (e != cudaSuccess) return c->cuda_fail(e, "window_select launch");

    // The top-k selection needs only the windowed medians: it runs beside the fleet baseline (on the
    // internal stream, behind the window medians); its scores, which need the baseline, are filled in by
    // the score pass.
    const bool want_topk = c->K > 0 && (d_topk_idx || d_topk_score);
    bool topk_side = false;
    if (want_topk) {
        TopkArgs t{};
        t.R = c->R;
        t.M = c->M;
        t.K = c->K;
        t.wmed = c->wmed(q);
        t.fleet_med = c->fleet_med();
        t.fleet_mad = c->fleet_mad();
        t.cand = c->topk_cand();
        t.ticket = c->ticket();
        t.idx = d_topk_idx;
        t.idx_keep = c->topk_idx(q);
        t.score = nullptr;
        // evaluations a few steps apart: the previous evaluation's threshold pre-selects the candidates
        if (c->sliding && gap <= kIncMaxNew) {
            t.hint = (TopkHint *)(c->ws + c->L.topk_hint);
            t.hcand = (unsigned long long *)(c->ws + c->L.topk_hint + 256);
        }
        // a deferred evaluation with a hinted (short) selection keeps it on the tail stream: two event calls less, and
        // the internal stream is free for the next evaluation's window medians
        if (c->overlap && !(defer && t.hint) && c->ensure_side()) {
            if (!(defer || forked)) {   // the window medians ran on `st`: order the internal stream behind them
                e = cudaEventRecord(c->ev_fork, st);
                if (e == cudaSuccess) e = cudaStreamWaitEvent(c->side, c->ev_fork, 0);
            }
            // deferred: on a stream of its own behind the window medians (ev_w), so that the next evaluation's window
            // medians need not queue behind it
            cudaStream_t tk = (defer && c->aux) ? c->aux : c->side;
            if (e == cudaSuccess && tk == c->aux) e = cudaStreamWaitEvent(c->aux, c->ev_w, 0);
            if (e == cudaSuccess) e = launch_topk(t, c->p, tk);
            if (e == cudaSuccess) e = cudaEventRecord(c->ev_topk, tk);
            topk_side = true;
        } else {
            e = launch_topk(t, c->p, ts);
        }
        if (e != cudaSuccess) return c->cuda_fail(e, "topk launch");
        c->launches += t.hint ? 2 : 1;
    }

    XrankArgs x{};
    x.base = c->wmed(q);
    x.row_stride = (long long)row;
    x.first_slot = 0;
    x.capacity = 1;
    x.R = c->R;
    x.M = c->M;
    x.med = c->fleet_med();
    x.mad = c->fleet_mad();
    x.med_user = d_fleet_med;
    x.mad_user = d_fleet_mad;
    x.status = c->status();
    e = c->xrank(x, 1, ts, !defer, 1);
    if (e != cudaSuccess) return c->cuda_fail(e, "fleet baseline launch");

    ScoreArgs s{};
    s.R = c->R;
    s.M = c->M;
    s.wmed = c->wmed(q);
    s.fleet_med = c->fleet_med();
    s.fleet_mad = c->fleet_mad();
    s.mask_base = c->mask();
    s.mask_bytes = c->mask_bytes();
    s.capacity = c->C;
    s.last_slot = last;
    s.n = n;
    s.consec = c->consec();
    s.scores = d_scores;
    s.counts = d_counts;
    s.metric_mask = d_metric_mask;
    s.flags = d_flags;
    s.tier = d_tier;
    s.flags_keep = c->lastflag();
    s.tier_keep = c->lasttier();
    // k-of-W counts slide like the window medians: the previous evaluation's counts plus / minus the exceedance
    // rows of the steps that entered / left (the rows that left must still be in the exceedance ring)
    s.kcnt = (uint16_t *)(c->ws + c->L.kcnt);
    {
        const long long p1 = c->cnt_seen, p0 = p1 - c->cnt_n, q1 = c->seen, q0 = q1 - n;
        if (c->sliding && p1 >= 0 && q0 < p1 && q1 - p1 <= kIncMaxNew && q0 - p0 <= kIncMaxNew && q1 - p0 <= c->C) {
            s.slide = 1;
            s.entering = (int)(q1 - p1);
            s.leaving = (int)(q0 - p0);
        }
        c->cnt_seen = c->seen;
        c->cnt_n = n;
    }
    s.topk_idx = want_topk ? c->topk_idx(q) : nullptr;
    s.topk_score = want_topk ? d_topk_score : nullptr;
    s.K = c->K;
    if (topk_side) {
        e = cudaStreamWaitEvent(ts, c->ev_topk, 0);
        if (e != cudaSuccess) return c->cuda_fail(e, "topk join");
    }
    e = launch_score_flag(s, c->p, ts);
    if (e != cudaSuccess) return c->cuda_fail(e, "score_flag launch");
    c->evals += 1;
    c->launches += 1 + window_launch_count(w) + (use_inc ? 1 : 0);
    if (defer) {
        e = cudaEventRecord(c->ev_e[q], c->tail);
        if (e != cudaSuccess) return c->cuda_fail(e, "event record");
        c->pending = true;
        // the sliding updates also read the steps that just left the window
        c->pending_n = n + ((use_inc ? ia.leaving : 0) > s.leaving ? (use_inc ? ia.leaving : 0) : s.leaving);
        c->pending_seen = c->seen;
        c->last_q = q;
        c->infl[q].on = true;
        c->infl[q].seen = c->seen;
        c->infl[q].n = c->pending_n;
    }
    return GUARD_OK;
}

size_t guard_sweep_workspace_bytes(int gpus, int reps, int metrics) {
    if (gpus < 1 || reps < 1 || reps > GUARD_MAX_WINDOW || metrics < 1 || metrics > GUARD_MAX_METRICS ||
        (long long)gpus * metrics > 0x7FFFFFFFLL)
        return 0;
    // fleet statistics, per-GPU medians, then the thread path's list of unserved series and its counter
    return align_up(3 * kMaxMetrics * sizeof(float)) + align_up((size_t)gpus * metrics * sizeof(float)) +
           align_up((size_t)gpus * metrics * sizeof(uint32_t)) + align_up(64);
}

int guard_sweep_qualify(const float *d_S, int nodes, int gpus_per_node, int reps, int metrics, const guard_thresholds *th,
                        int32_t pct_ppm, void *d_workspace, size_t workspace_bytes, float *d_gpu_med, float *d_fleet_med,
                        float *d_fleet_mad, float *d_fleet_cut, uint32_t *d_fail_mask, uint8_t *d_gpu_pass,
                        uint8_t *d_node_pass, uint32_t *d_status, void *stream) {
    if (!d_S || nodes < 1 || gpus_per_node < 1 || (long long)nodes * gpus_per_node > 0x7FFFFFFFLL) {
        set_error(g_error, "d_S is NULL or nodes / gpus_per_node out of range");
        return GUARD_ERR_ARG;
    }
    const int G = nodes * gpus_per_node;
    const size_t need = guard_sweep_workspace_bytes(G, reps, metrics);
    if (need == 0) { set_error(g_error, "invalid sweep sizes"); return GUARD_ERR_ARG; }
    if (pct_ppm < 0 || pct_ppm > 1000000) { set_error(g_error, "pct_ppm must be in 0..1000000"); return GUARD_ERR_ARG; }
    MetricParams p;
    if (const char *msg = fill_params(p, th, metrics, 1, false)) { set_error(g_error, "%s", msg); return GUARD_ERR_ARG; }
    if (!d_workspace || ((uintptr_t)d_workspace % kAlign) != 0 || workspace_bytes < need) {
        set_error(g_error, "sweep workspace must be non-NULL, 256-byte aligned and at least %zu bytes", need);
        return GUARD_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)stream;
    float *fleet = (float *)d_workspace;
    float *gmed = (float *)((char *)d_workspace + align_up(3 * kMaxMetrics * sizeof(float)));

    SweepMedArgs sm{};
    sm.S = d_S;
    sm.G = G;
    sm.reps = reps;
    sm.M = metrics;
    sm.gmed = gmed;
    sm.gmed_user = d_gpu_med;
    sm.status = d_status;
    sm.list = (uint32_t *)((char *)gmed + align_up((size_t)G * metrics * sizeof(float)));
    sm.list_count = (uint32_t *)((char *)sm.list + align_up((size_t)G * metrics * sizeof(uint32_t)));
    cudaError_t e = launch_sweep_medians(sm, st);
    if (e != cudaSuccess) { set_error(g_error, "sweep medians launch: %s", cudaGetErrorString(e)); return GUARD_ERR_CUDA; }

    // nearest-rank percentile of the bad tail: the j-th worst of G values
    long long j = ((long long)pct_ppm * G + 999999) / 1000000;
    if (j < 1) j = 1;
    if (j > G) j = G;
    XrankArgs x{};
    x.base = gmed;
    x.row_stride = (long long)G * metrics;
    x.first_slot = 0;
    x.capacity = 1;
    x.R = G;
    x.M = metrics;
    x.med = fleet;
    x.mad = fleet + kMaxMetrics;
    x.cut = fleet + 2 * kMaxMetrics;
    x.med_user = d_fleet_med;
    x.mad_user = d_fleet_mad;
    for (int m = 0; m < metrics; ++m) x.cut_rank[m] = p.dir[m] < 0 ? (int)(j - 1) : (int)(G - j);
    x.status = d_status;
    e = xrank_column_supported(G) ? launch_xrank_column(x, p, 1, st) : launch_xrank_direct(x, p, 1, st);
    if (e != cudaSuccess) { set_error(g_error, "sweep fleet statistics launch: %s", cudaGetErrorString(e)); return GUARD_ERR_CUDA; }
    if (d_fleet_cut) {
        e = cudaMemcpyAsync(d_fleet_cut, fleet + 2 * kMaxMetrics, metrics * sizeof(float), cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) { set_error(g_error, "cudaMemcpyAsync: %s", cudaGetErrorString(e)); return GUARD_ERR_CUDA; }
    }
    SweepVerdictArgs v{};
    v.nodes = nodes;
    v.gpus_per_node = gpus_per_node;
    v.M = metrics;
    v.gmed = gmed;
    v.fleet_med = fleet;
    v.fleet_mad = fleet + kMaxMetrics;
    v.fleet_cut = fleet + 2 * kMaxMetrics;
    v.fail_mask = d_fail_mask;
    v.gpu_pass = d_gpu_pass;
    v.node_pass = d_node_pass;
    e = launch_sweep_verdict(v, p, st);
    if (e != cudaSuccess) { set_error(g_error, "sweep verdict launch: %s", cudaGetErrorString(e)); return GUARD_ERR_CUDA; }
    return GUARD_OK;
}

int guard_node_verdict(guard_ctx *c, uint8_t *d_node_flag, uint8_t *d_node_tier, uint16_t *d_node_stall, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    if (c->R % c->ranks_per_node != 0)
        return c->fail(GUARD_ERR_ARG, "ranks (%d) is not a multiple of ranks_per_node (%d)", c->R, c->ranks_per_node);
    if (c->evals < 1 || c->seen_at_eval != c->seen)
        return c->fail(GUARD_ERR_NOT_READY, "guard_node_verdict must follow guard_score with no ingest in between");
    NodeArgs a{};
    a.R = c->R;
    a.ranks_per_node = c->ranks_per_node;
    a.nodes = c->R / c->ranks_per_node;
    a.primary = c->p.primary;
    a.flags = c->lastflag();
    a.tier = c->lasttier();
    a.mask_base = c->mask();
    a.mask_bytes = c->mask_bytes();
    a.capacity = c->C;
    a.last_slot = (int)((c->seen - 1) % c->C);
    a.n = (int)(c->seen < c->W ? c->seen : c->W);
    a.node_flag = d_node_flag;
    a.node_tier = d_node_tier;
    a.node_stall = d_node_stall;
    // a deferred evaluation still pending: the fold joins it on the evaluation's own stream
    const bool on_tail = c->pending && c->tail;
    cudaStream_t ts = on_tail ? c->tail : (cudaStream_t)stream;
    cudaError_t e = launch_node_verdict(a, ts);
    if (e == cudaSuccess && on_tail) e = cudaEventRecord(c->ev_e[c->last_q], c->tail);
    if (e != cudaSuccess) return c->cuda_fail(e, "node verdict launch");
    c->launches += 1;
    return GUARD_OK;
}

// ---- state export / import -----------------------------------------------------------------------
namespace {
struct StateHeader {
    uint32_t magic, version;
    int32_t R, M, W, k, K, mask_bytes;
    int64_t seen, evals, seen_at_eval;
    int32_t steps;      // ring steps stored: min(seen, W)
    int32_t inc_n;      // sliding-window state: window length it is current for
    int64_t inc_seen;   // ... and the step count (-1: none)
    int32_t hints_ready, pad;
};
constexpr uint32_t kStateMagic = 0x47524453u;   // "GRDS"
constexpr size_t kStateHeaderBytes = 256;

struct StateLayout { size_t status, fleet, consec, lastflag, lasttier, wmed, wspread, wcentre, inc, mask, ring, total; };
StateLayout state_layout(const guard_ctx *c) {
    StateLayout s{};
    const size_t RM = (size_t)c->R * c->M * sizeof(float);
    size_t off = kStateHeaderBytes;
    s.status = off;   off = align_up(off + 64);
    s.fleet = off;    off = align_up(off + 3 * kMaxMetrics * sizeof(float));
    s.consec = off;   off = align_up(off + (size_t)c->R);
    s.lastflag = off; off = align_up(off + (size_t)c->R);
    s.lasttier = off; off = align_up(off + (size_t)c->R);
    s.wmed = off;     off = align_up(off + RM);
    s.wspread = off;  off = align_up(off + RM);
    s.wcentre = off;  off = align_up(off + RM);
    s.inc = off;      off = align_up(off + (3 + kIncSlots) * window_inc_bytes(c->R * c->M));
    s.mask = off;     off = align_up(off + (size_t)c->W * c->R * c->mask_bytes());
    s.ring = off;     off = align_up(off + (size_t)c->W * RM);
    s.total = off;
    return s;
}

// Copies the last `steps` ring rows (row_bytes each) between the ring at `ring` (capacity C, newest
// row at step index seen - 1) and a compact buffer holding them oldest first.
cudaError_t copy_rows(char *ring, char *compact, size_t row_bytes, long long seen, int steps, int C, bool to_compact,
                      cudaStream_t st) {
    long long step = seen - steps;
    int done = 0;
    while (done < steps) {
        const int slot = (int)((step + done) % C);
        const int run = (steps - done < C - slot) ? (steps - done) : (C - slot);
        char *r = ring + (size_t)slot * row_bytes, *q = compact + (size_t)done * row_bytes;
        cudaError_t e = cudaMemcpyAsync(to_compact ? q : r, to_compact ? r : q, (size_t)run * row_bytes, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return e;
        done += run;
    }
    return cudaSuccess;
}
}  // namespace

size_t guard_state_bytes(const guard_ctx *c) { return c ? state_layout(c).total : 0; }

int guard_state_export(guard_ctx *c, void *d_state, size_t state_bytes, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    const StateLayout sl = state_layout(c);
    if (!d_state || ((uintptr_t)d_state % 16) != 0 || state_bytes < sl.total)
        return c->fail(GUARD_ERR_WORKSPACE, "state buffer must be non-NULL, 16-byte aligned and at least %zu bytes", sl.total);
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = c->join(st);
    if (e == cudaSuccess) e = c->join_xs(st);
    if (e != cudaSuccess) return c->cuda_fail(e, "join of deferred work");
    char *d = (char *)d_state;
    const size_t RM = (size_t)c->R * c->M * sizeof(float);
    StateHeader h{};
    h.magic = kStateMagic; h.version = 1;
    h.R = c->R; h.M = c->M; h.W = c->W; h.k = c->k; h.K = c->K; h.mask_bytes = c->mask_bytes();
    h.seen = c->seen; h.evals = c->evals; h.seen_at_eval = c->seen_at_eval;
    h.steps = (int)(c->seen < c->W ? c->seen : c->W);
    h.inc_n = c->inc_n; h.inc_seen = c->inc_seen; h.hints_ready = c->hints_ready ? 1 : 0;
    // pageable host source: the runtime stages it before the call returns
    e = cudaMemcpyAsync(d, &h, sizeof(h), cudaMemcpyHostToDevice, st);
    auto dd = [&](size_t dst_off, const void *src, size_t n) {
        if (e == cudaSuccess) e = cudaMemcpyAsync(d + dst_off, src, n, cudaMemcpyDeviceToDevice, st);
    };
    dd(sl.status, c->status(), 64);
    dd(sl.fleet, c->fleet_med(), 3 * kMaxMetrics * sizeof(float));
    dd(sl.consec, c->consec(), (size_t)c->R);
    dd(sl.lastflag, c->lastflag(), (size_t)c->R);
    dd(sl.lasttier, c->lasttier(), (size_t)c->R);
    dd(sl.wmed, c->wmed(c->prev_q()), RM);   // the medians of the evaluation made last
    dd(sl.wspread, c->ws + c->L.wspread, RM);
    dd(sl.wcentre, c->ws + c->L.wcentre, RM);
    {   // sliding-window state: four arrays, stored back to back
        const size_t ib = window_inc_bytes(c->R * c->M);
        dd(sl.inc, c->ws + c->L.inc_lo, ib);
        dd(sl.inc + ib, c->ws + c->L.inc_hi, ib);
        dd(sl.inc + 2 * ib, c->ws + c->L.inc_cnt, ib);
        dd(sl.inc + 3 * ib, c->ws + c->L.inc_val, kIncSlots * ib);
    }
    if (e == cudaSuccess) e = copy_rows((char *)c->mask(), d + sl.mask, (size_t)c->R * c->mask_bytes(), c->seen, h.steps, c->C, true, st);
    if (e == cudaSuccess) e = copy_rows((char *)c->ring(), d + sl.ring, RM, c->seen, h.steps, c->C, true, st);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_state_export");
    return GUARD_OK;
}

int guard_state_import(guard_ctx *c, const void *d_state, size_t state_bytes, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    const StateLayout sl = state_layout(c);
    if (!d_state || ((uintptr_t)d_state % 16) != 0 || state_bytes < sl.total)
        return c->fail(GUARD_ERR_WORKSPACE, "state buffer must be non-NULL, 16-byte aligned and at least %zu bytes", sl.total);
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = c->join(st);
    if (e == cudaSuccess) e = c->join_xs(st);
    StateHeader h{};
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, d_state, sizeof(h), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_state_import");
    if (h.magic != kStateMagic || h.version != 1) return c->fail(GUARD_ERR_ARG, "not a state written by guard_state_export");
    if (h.R != c->R || h.M != c->M || h.W != c->W || h.k != c->k || h.K != c->K || h.mask_bytes != c->mask_bytes())
        return c->fail(GUARD_ERR_ARG, "state was exported from a context of other sizes (ranks %d metrics %d W %d k %d topk %d)",
                       h.R, h.M, h.W, h.k, h.K);
    if (h.seen < 0 || h.steps != (int)(h.seen < h.W ? h.seen : h.W) || h.evals < 0 || h.seen_at_eval > h.seen ||
        h.inc_seen > h.seen || h.inc_n < 0 || h.inc_n > h.W)
        return c->fail(GUARD_ERR_ARG, "state header is inconsistent");
    const char *d = (const char *)d_state;
    const size_t RM = (size_t)c->R * c->M * sizeof(float);
    // scratch that must start at zero (ticket, bracketed-path flags) is cleared with the rest of the prefix
    e = cudaMemsetAsync(c->ws, 0, c->L.wmed, st);
    auto dd = [&](void *dst, size_t src_off, size_t n) {
        if (e == cudaSuccess) e = cudaMemcpyAsync(dst, d + src_off, n, cudaMemcpyDeviceToDevice, st);
    };
    dd(c->status(), sl.status, 64);
    dd(c->fleet_med(), sl.fleet, 3 * kMaxMetrics * sizeof(float));
    dd(c->consec(), sl.consec, (size_t)c->R);
    dd(c->lastflag(), sl.lastflag, (size_t)c->R);
    dd(c->lasttier(), sl.lasttier, (size_t)c->R);
    dd(c->wmed((int)((h.evals + 1) & 1)), sl.wmed, RM);   // where the next evaluation looks for the previous medians
    dd(c->ws + c->L.wspread, sl.wspread, RM);
    dd(c->ws + c->L.wcentre, sl.wcentre, RM);
    {
        const size_t ib = window_inc_bytes(c->R * c->M);
        dd(c->ws + c->L.inc_lo, sl.inc, ib);
        dd(c->ws + c->L.inc_hi, sl.inc + ib, ib);
        dd(c->ws + c->L.inc_cnt, sl.inc + 2 * ib, ib);
        dd(c->ws + c->L.inc_val, sl.inc + 3 * ib, kIncSlots * ib);
    }
    if (e == cudaSuccess) e = copy_rows((char *)c->mask(), const_cast<char *>(d) + sl.mask, (size_t)c->R * c->mask_bytes(), h.seen, h.steps, c->C, false, st);
    if (e == cudaSuccess) e = copy_rows((char *)c->ring(), const_cast<char *>(d) + sl.ring, RM, h.seen, h.steps, c->C, false, st);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_state_import");
    c->seen = h.seen;
    c->evals = h.evals;
    c->seen_at_eval = h.seen_at_eval;
    c->inc_seen = h.inc_seen;
    c->inc_n = h.inc_n;
    c->cnt_seen = -1;   // the kept counts are not part of the state: the next evaluation recounts
    c->hints_ready = h.hints_ready != 0;
    c->new_epoch();   // the split scratch describes other data
    c->fork_fresh = false;
    return GUARD_OK;
}

int guard_debug_set_wait_limit(guard_ctx *c, long long cycles) {
    if (!c || cycles < 0) return GUARD_ERR_ARG;
    c->wait_limit = cycles;
    return GUARD_OK;
}

int guard_sync_status(guard_ctx *c, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    uint32_t s = 0;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&s, c->status(), sizeof(s), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_sync_status");
    const int code = status_to_code(s);
    if (code != GUARD_OK) c->fail(code, "device status word 0x%x", s);
    return code;
}

int guard_reset(guard_ctx *c, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws, 0, c->L.wmed, (cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "cudaMemsetAsync");
    c->seen = 0;
    c->evals = 0;
    c->seen_at_eval = 0;
    c->inc_seen = -1;
    c->cnt_seen = -1;
    c->hints_ready = false;
    c->new_epoch();
    return GUARD_OK;
}

int guard_profile_enable(guard_ctx *c, int on) {
    if (!c) return GUARD_ERR_ARG;
    c->profiling = on;
    if (!on) {
        for (auto &pr : c->prof) { cudaEventDestroy(pr.first); cudaEventDestroy(pr.second); }
        c->prof.clear();
    }
    return GUARD_OK;
}

int guard_profile_read(guard_ctx *c, double *total_ms, int64_t *launches) {
    if (!c || !total_ms || !launches) return GUARD_ERR_ARG;
    double sum = 0.0;
    for (auto &pr : c->prof) {
        cudaError_t e = cudaEventSynchronize(pr.second);
        float ms = 0.0f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, pr.first, pr.second);
        if (e != cudaSuccess) return c->cuda_fail(e, "guard_profile_read");
        sum += ms;
        cudaEventDestroy(pr.first);
        cudaEventDestroy(pr.second);
    }
    *total_ms = sum;
    *launches = (int64_t)c->prof.size();
    c->prof.clear();
    return GUARD_OK;
}

int64_t guard_steps_seen(const guard_ctx *c) { return c ? c->seen : 0; }

int64_t guard_kernel_launches(const guard_ctx *c) { return c ? c->launches : 0; }

int guard_fallback_reasons(guard_ctx *c, uint32_t out[6], void *stream) {
    if (!c || !out) return GUARD_ERR_ARG;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out, c->status() + 2, 6 * sizeof(uint32_t), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_fallback_reasons");
    return GUARD_OK;
}

int guard_window_fallbacks(guard_ctx *c, uint32_t out[6], void *stream) {
    if (!c || !out) return GUARD_ERR_ARG;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out, c->status() + 8, 6 * sizeof(uint32_t), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_window_fallbacks");
    return GUARD_OK;
}

int64_t guard_sliding_rebuilds(guard_ctx *c, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    uint32_t n = 0;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&n, c->status() + 14, sizeof(n), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_sliding_rebuilds");
    return (int64_t)n;
}

int64_t guard_fallback_steps(guard_ctx *c, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    uint32_t n = 0;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&n, c->status() + 1, sizeof(n), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_fallback_steps");
    return (int64_t)n;
}

int guard_set_sliding(guard_ctx *c, int on) {
    if (!c) return GUARD_ERR_ARG;
    c->sliding = on != 0;
    return GUARD_OK;
}

int guard_set_row_hints(guard_ctx *c, int on) {
    if (!c) return GUARD_ERR_ARG;
    c->row_hints = on != 0;
    return GUARD_OK;
}

int guard_row_hints(guard_ctx *c, uint32_t out[6], void *stream) {
    if (!c || !out) return GUARD_ERR_ARG;
    for (int i = 0; i < 6; ++i) out[i] = 0;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = c->join(st);
    if (e == cudaSuccess) e = c->join_xs(st);
    for (int site = 0; site < 2 && e == cudaSuccess && c->L.xr_gridp; ++site)   // rows and settled are the first two words
        e = cudaMemcpyAsync(&out[2 * site], c->hint_state(site), 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess)   // hits and misses of the hinted top-k pass
        e = cudaMemcpyAsync(&out[4], (char *)(c->ws + c->L.topk_hint) + offsetof(TopkHint, hits), 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_row_hints");
    return GUARD_OK;
}

int guard_set_deferred(guard_ctx *c, int on) {
    if (!c) return GUARD_ERR_ARG;
    c->deferred = on != 0;
    return GUARD_OK;
}

int guard_join(guard_ctx *c, void *stream) {
    if (!c) return GUARD_ERR_ARG;
    cudaError_t e = c->join((cudaStream_t)stream);
    if (e == cudaSuccess) e = c->join_xs((cudaStream_t)stream);
    if (e != cudaSuccess) return c->cuda_fail(e, "guard_join");
    return GUARD_OK;
}

int guard_set_overlap(guard_ctx *c, int on) {
    if (!c) return GUARD_ERR_ARG;
    c->overlap = on != 0;
    c->fork_fresh = false;
    return GUARD_OK;
}

void guard_destroy(guard_ctx *c) {
    if (c) {
        guard_profile_enable(c, 0);
        for (int k = 0; k < kIngestStreams; ++k)
            if (c->xs[k]) {
                cudaStreamSynchronize(c->xs[k]);
                cudaStreamDestroy(c->xs[k]);
                cudaEventDestroy(c->ev_xs[k]);
            }
        if (c->ev_data) cudaEventDestroy(c->ev_data);
        if (c->tail) {
            cudaStreamSynchronize(c->tail);
            cudaStreamDestroy(c->tail);
            if (c->aux) { cudaStreamSynchronize(c->aux); cudaStreamDestroy(c->aux); }
            cudaEventDestroy(c->ev_x);
            cudaEventDestroy(c->ev_w);
            cudaEventDestroy(c->ev_e[0]);
            cudaEventDestroy(c->ev_e[1]);
        }
        if (c->side) {
            cudaStreamDestroy(c->side);
            cudaEventDestroy(c->ev_fork);
            cudaEventDestroy(c->ev_join);
            if (c->ev_topk) cudaEventDestroy(c->ev_topk);
        }
    }
    delete c;
}

const char *guard_last_error(const guard_ctx *c) { return c ? c->error : g_error; }

uint32_t guard_key_from_float(float x) {
    uint32_t b;
    memcpy(&b, &x, 4);
    return key_of_bits(b);
}

float guard_float_from_key(uint32_t key) {
    const uint32_t b = bits_of_key(key);
    float x;
    memcpy(&x, &b, 4);
    return x;
}

}  // extern "C"
