/*
 * guard_b200.h -- C ABI of the straggler-scoring library for NVIDIA B200 (sm_100a).
 *
 * The library computes the numerical core of Guard's online monitor (paper Section 4.2,
 * "Online Monitoring Strategy") and the scoring half of its offline node sweep
 * (Sections 5.2-5.4) over a fleet telemetry tensor T[step, rank, metric], float32,
 * metric innermost, row-major.  The paper fixes the rules in words (peer-relative
 * evaluation, several indicators, deviation sustained over evaluation windows, step time
 * as the primary signal, response tiers at about 10 % and at 20 % or more, a node passes
 * only if every part of its sweep passes) and names no statistic; the statistics below
 * (median, raw median absolute deviation, the 0.6745-scaled robust z with a one-sided
 * cut-off, k-of-W persistence, nearest-rank percentile) are the reading this library
 * implements.
 *
 * Conventions
 *   - Every pointer whose name starts with d_ is DEVICE memory owned by the caller; all
 *     other pointers are HOST memory.  The library never allocates, frees or keeps device
 *     memory of its own: the caller hands it one workspace (guard_workspace_bytes) that
 *     holds the telemetry ring and all state, and must keep it alive and untouched until
 *     guard_destroy.
 *   - `stream` is a cudaStream_t passed as void*.  All work is ordered on it.  The calls that
 *     synchronise `stream` with the host are the ones that hand a value back from the device:
 *     guard_sync_status, guard_fallback_steps, guard_fallback_reasons, guard_window_fallbacks,
 *     guard_sliding_rebuilds, guard_row_hints and guard_state_import;
 *     guard_profile_read waits for the events it recorded.  No other call synchronises.
 *     (guard_score may run the window medians on an internal stream forked from and joined back
 *     into `stream` with events, so that they overlap the preceding guard_ingest; to the caller
 *     everything behaves as if enqueued on `stream`.  guard_set_overlap(ctx, 0) turns that off.)
 *     Calls on one context must be issued in order on streams that are ordered with respect to
 *     each other.
 *   - Every function returns a status (GUARD_OK = 0, errors negative) and never throws,
 *     aborts or traps.  Argument errors are detected on the host before anything is
 *     enqueued.  Data-dependent errors (non-finite telemetry, a bounded wait that ran out)
 *     are recorded in a sticky device status word that guard_sync_status reads back.
 *   - Output pointers documented as "or NULL" may be NULL to skip that output.
 *   - Order of values is the IEEE total order of finite float32 (so -0 < +0).  All
 *     decisions (exceedance, flag, tier, percentile cut, top-k order) use single float32
 *     subtract / multiply / fabs / compare only and are reproducible bit for bit;
 *     reported scores use one extra float32 division.
 */
#ifndef GUARD_B200_H
#define GUARD_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GUARD_MAX_METRICS 32
#define GUARD_MAX_TOPK 1024
#define GUARD_MAX_WINDOW 65535

enum {
    GUARD_OK = 0,
    GUARD_ERR_ARG = -1,        /* invalid argument (see guard_last_error) */
    GUARD_ERR_WORKSPACE = -2,  /* workspace NULL, misaligned (256 B) or too small */
    GUARD_ERR_NOT_READY = -3,  /* guard_score before the first ingested step */
    GUARD_ERR_NONFINITE = -4,  /* NaN or Inf seen in ingested telemetry (sticky) */
    GUARD_ERR_TIMEOUT = -5,    /* a bounded on-device wait ran out (sticky) */
    GUARD_ERR_CUDA = -6,       /* a CUDA runtime call failed */
    GUARD_ERR_INTERNAL = -7    /* a device-side consistency check failed (sticky) */
};

typedef struct guard_ctx guard_ctx; /* host object; owns no device memory */

/* Detector parameters; copied by guard_create / guard_sweep_qualify (host memory). */
typedef struct {
    int32_t primary;        /* index of the primary metric: training-step time (Sec. 4.2) */
    int32_t min_signals;    /* metrics that must deviate persistently, "multiple" (Sec. 4.2); clipped to M */
    int32_t n_consec;       /* consecutive evaluations required before a flag is raised (>= 1) */
    int32_t ranks_per_node; /* >= 1; 8 in the paper's cluster (Sec. 7.1): group size of guard_node_verdict */
    float tier_moderate;    /* relative slowdown of the moderate tier, 0.10 (Sec. 4.2) */
    float tier_severe;      /* relative slowdown of the severe tier, 0.20 (Sec. 4.2) */
    const int8_t *dir;      /* [M] +1: larger is worse (durations, temperature); -1: smaller is worse */
    const float *thr;       /* [M] robust-z cut-off, e.g. 3.5 */
    const float *floor_rel; /* [M] floor of the spread relative to |median|, e.g. 1e-4 */
    const float *floor_abs; /* [M] absolute floor of the spread, e.g. 0 */
} guard_thresholds;

/* Bytes of device workspace needed by a context with these sizes (0 on invalid sizes).
 * The ring holds capacity_steps steps; windows use the last min(W, seen) of them. */
size_t guard_workspace_bytes(int ranks, int metrics, int W, int capacity_steps, int topk);

/*
 * Create a context for `ranks` peers and `metrics` (1..32) indicators, window W
 * (1..65535 steps), persistence k (1..W): a metric is persistent for a rank when at
 * least k of the last W steps exceeded the per-step peer baseline (the temporal filter of
 * Sec. 4.2).  topk in 0..min(ranks, 1024).
 * d_workspace: device memory, 256-byte aligned, >= guard_workspace_bytes(...); its state
 * part is zeroed on `stream`.  Errors: GUARD_ERR_ARG, GUARD_ERR_WORKSPACE, GUARD_ERR_CUDA.
 */
int guard_create(guard_ctx **out, int ranks, int metrics, int W, int k, const guard_thresholds *th,
                 int capacity_steps, int topk, void *d_workspace, size_t workspace_bytes, void *stream);

/*
 * Where the next `steps` steps of telemetry go inside the ring, for producers that write
 * telemetry in place (a gather kernel, a host-to-device copy): *d_slot receives a device
 * pointer to steps*ranks*metrics contiguous floats.  Fails with GUARD_ERR_ARG if that
 * span would wrap around the end of the ring (choose capacity_steps as a multiple of the
 * block size).  Passing the returned pointer to guard_ingest skips the copy into the ring.
 */
int guard_ring_reserve(guard_ctx *ctx, int steps, float **d_slot);

/*
 * Ingest B (1..capacity_steps) steps: d_block[B][ranks][metrics] float32.  Appends them
 * to the ring (a device-to-device copy unless d_block came from guard_ring_reserve) and
 * computes, for every step and metric, the cross-rank median and raw MAD -- the peer
 * baseline of that step (Sec. 4.2, evaluation "relative to peer nodes") -- and the
 * one-sided exceedance bit of every rank,
 *     dir * (x - med) > (float)(thr / 0.6745) * max(mad, floor_rel * |med|, floor_abs),
 * stored in the exceedance ring.  Even rank counts use the midpoint of the two middle
 * values (one float32 add, one multiply by 0.5).
 * d_step_med, d_step_mad: [B][metrics] float32 or NULL.
 * Non-finite input sets the sticky GUARD_ERR_NONFINITE status; results are then
 * unspecified until guard_reset.
 */
int guard_ingest(guard_ctx *ctx, const float *d_block, int B, float *d_step_med, float *d_step_mad, void *stream);

/*
 * One evaluation over the window of the last n = min(W, seen) steps (Sec. 4.2):
 *   d_wmed[r][m]    windowed per-rank median (blind to isolated spikes)
 *   d_fleet_med[m], d_fleet_mad[m]  cross-rank median / raw MAD of the windowed medians
 *   d_scores[r][m]  0.6745 * dir * (wmed - fleet_med) / scale, 0 where wmed == fleet_med
 *   d_counts[r][m]  exceedances among the window's steps (k-of-W persistence filter)
 *   d_metric_mask[r] bit m set when the windowed median exceeds the cut-off AND count >= k
 *   d_flags[r]      1 when the primary metric's bit is set, at least min_signals bits are
 *                   set, and this held for n_consec consecutive evaluations
 *   d_tier[r]       3: flagged and primary slowdown >= tier_severe * |fleet_med|;
 *                   2: flagged and >= tier_moderate; 1: some bit set ("pending
 *                   verification"); 0 otherwise
 *   d_topk_idx[K], d_topk_score[K]  the K ranks with the largest dir * wmed of the primary
 *                   metric (ties: lower rank first) and their primary scores
 * Every output is "or NULL".  Updates the per-rank consecutive-evaluation counters.
 * Errors: GUARD_ERR_NOT_READY before the first step.
 */
int guard_score(guard_ctx *ctx, float *d_wmed, float *d_fleet_med, float *d_fleet_mad, float *d_scores,
                uint16_t *d_counts, uint32_t *d_metric_mask, uint8_t *d_flags, uint8_t *d_tier,
                int32_t *d_topk_idx, float *d_topk_score, void *stream);

/* Bytes of device workspace needed by guard_sweep_qualify (0 on invalid sizes). */
size_t guard_sweep_workspace_bytes(int gpus, int reps, int metrics);

/*
 * Offline node-sweep qualification (Sec. 5.2-5.4): d_S[g][rep][metric] float32 holds the
 * repeated benchmark results of GPU g = node * gpus_per_node + local index.  Per GPU and
 * metric the median over the repetitions; per metric over all GPUs the median, raw MAD
 * and the nearest-rank percentile cut of the bad tail (j = ceil(pct_ppm * G / 1e6)
 * clipped to [1, G]; the j-th worst value).  Metric m fails GPU g when it is a robust-z
 * outlier in the bad direction AND strictly beyond the cut.  A GPU passes when no metric
 * fails; a node passes when all its GPUs pass (the pass rule of Sec. 5.4).
 * th->dir/thr/floor_rel/floor_abs are used; the other
 * fields are ignored.  Outputs ("or NULL"): d_gpu_med[G][M], d_fleet_med/mad/cut[M],
 * d_fail_mask[G], d_gpu_pass[G], d_node_pass[nodes].  d_status: device uint32 or NULL,
 * receives sticky status bits (1 = non-finite input, 2 = wait ran out, 4 = internal).
 */
int guard_sweep_qualify(const float *d_S, int nodes, int gpus_per_node, int reps, int metrics,
                        const guard_thresholds *th, int32_t pct_ppm, void *d_workspace, size_t workspace_bytes,
                        float *d_gpu_med, float *d_fleet_med, float *d_fleet_mad, float *d_fleet_cut,
                        uint32_t *d_fail_mask, uint8_t *d_gpu_pass, uint8_t *d_node_pass, uint32_t *d_status,
                        void *stream);

/*
 * Top-k of an evaluation without any allocation.  (The paper has no counterpart: this
 * entry point exists only for callers that cannot allocate device memory.)
 *
 * Some users of this library run as a telemetry sidecar next to a training job on the same
 * GPU.  There the job's own allocator has usually claimed the device memory up front, and
 * cudaMalloc / cudaFree synchronise the whole device, which would stall the job's streams;
 * such a caller cannot size and hand over a workspace just to re-rank a result.  This call
 * therefore takes its scratch from a fixed array inside the library image
 * (64 * GUARD_TOPK_STATIC_MAX_K candidate entries plus one ticket line = 131 328 bytes,
 * held by every GPU that loads the library until the process exits) and calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 * Inputs are the device arrays an evaluation produced (guard_score outputs or the
 * caller's own): d_wmed[ranks][metrics], d_fleet_med[metrics], d_fleet_mad[metrics];
 * th->primary, th->dir, th->floor_rel and th->floor_abs are used, the rest is ignored.
 * Outputs (either may be NULL): d_topk_idx[topk], d_topk_score[topk], identical to what
 * guard_score returns for the same inputs.
 * Limits: 1 <= topk <= min(ranks, GUARD_TOPK_STATIC_MAX_K), ranks <=
 * GUARD_TOPK_STATIC_MAX_RANKS; anything larger is rejected with GUARD_ERR_ARG and a text
 * in guard_last_error(NULL).
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call before starting any stream capture.
 * All calls on a device share the one array, which keeps the previous call's contents
 * (the call clears the ticket it needs at zero on `stream`): two calls whose kernels can
 * overlap on the GPU -- different streams, no ordering between them -- race on it.  Issue
 * them on one stream or order them with events.
 */
#define GUARD_TOPK_STATIC_MAX_K 256
#define GUARD_TOPK_STATIC_MAX_RANKS (1 << 24)
int guard_topk_static(const float *d_wmed, const float *d_fleet_med, const float *d_fleet_mad, int ranks, int metrics,
                      const guard_thresholds *th, int topk, int32_t *d_topk_idx, float *d_topk_score, void *stream);

/*
 * Node-level fold of the last evaluation.  The paper acts on nodes (Sec. 4.2: a flagged node
 * leaves the healthy pool; Sec. 7.1: 8 GPUs per node; the three response classes of
 * Sec. 4.2), so the per-rank results are folded over groups of ranks_per_node consecutive
 * ranks, nodes = ranks / ranks_per_node:
 *   d_node_flag[nodes]   1 when any rank of the node is flagged
 *   d_node_tier[nodes]   highest tier among its ranks: 0 none, 1 pending verification,
 *                        2 mitigate at the next checkpoint, 3 restart now
 *   d_node_stall[nodes]  steps of the evaluation's window in which EVERY rank of the node
 *                        exceeded the step's peer baseline on the primary metric at once
 *                        (a correlated whole-node stall, as opposed to one slow GPU)
 * Every output is "or NULL".  Must follow guard_score with no guard_ingest in between
 * (GUARD_ERR_NOT_READY otherwise); ranks must be a multiple of ranks_per_node
 * (GUARD_ERR_ARG).  After a deferred guard_score the fold becomes part of that pending
 * evaluation: its outputs are complete where the evaluation's are.
 */
int guard_node_verdict(guard_ctx *ctx, uint8_t *d_node_flag, uint8_t *d_node_tier, uint16_t *d_node_stall, void *stream);

/*
 * Checkpoint / resume of a context (the monitor of Sec. 4.2 runs for the months of a
 * training job and must survive its own restarts).  The state is the telemetry and the
 * exceedance bits of the last min(W, steps seen) steps, the consecutive-evaluation counters,
 * the last evaluation's medians, per-rank verdicts and search intervals, the status words
 * and the step / evaluation counters: everything later results depend on.
 * guard_state_bytes: size of the state of this context (fixed by its sizes).
 * guard_state_export: waits (on `stream`, not on the host) for deferred work, then copies the
 *   state into d_state (DEVICE memory, 16-byte aligned, >= guard_state_bytes).
 * guard_state_import: loads a state exported by a context of the same ranks, metrics, W, k and
 *   topk (capacity_steps may differ) into this context, replacing what it held; it reads the
 *   state's header back and therefore synchronises `stream`.  A context that imports and then
 *   sees the same steps gives bit-identical results to the one that never stopped.
 * Errors: GUARD_ERR_WORKSPACE (buffer NULL, misaligned or too small), GUARD_ERR_ARG (not a
 * state, or one of other sizes), GUARD_ERR_CUDA.
 */
size_t guard_state_bytes(const guard_ctx *ctx);
int guard_state_export(guard_ctx *ctx, void *d_state, size_t state_bytes, void *stream);
int guard_state_import(guard_ctx *ctx, const void *d_state, size_t state_bytes, void *stream);

/*
 * Repeat-offender rule of the triage workflow (Sec. 6: a node that enters triage three times
 * within a week is replaced instead of being triaged again).  Host-only bookkeeping, no GPU
 * work.  guard_triage_create: `nodes` node ids 0..nodes-1, `limit` entries (the paper: 3)
 * within `period_s` seconds (the paper: one week = 604800).  guard_triage_record: node
 * `node` enters triage at `time_s` (seconds, not before the node's previous entry); returns
 * 1 when this is at least the limit-th entry no more than period_s old (both ends counted),
 * i.e. the node is to be terminated, 0 when it goes through triage, GUARD_ERR_ARG on a bad
 * node id or a time that runs backwards.  *entries_in_period (or NULL) receives the number
 * of entries, this one included, inside that span, counted up to `limit`.
 */
typedef struct guard_triage guard_triage;
int guard_triage_create(guard_triage **out, int nodes, int limit, int64_t period_s);
int guard_triage_record(guard_triage *t, int node, int64_t time_s, int *entries_in_period);
void guard_triage_destroy(guard_triage *t);

/* Test hook: limit, in clock cycles, of the first wait for a staged tile in the warp-per-series
 * window kernel (0 restores the default of about a second).  With a limit of a few cycles that
 * wait runs out while the copies are still in flight; the kernel then records
 * GUARD_ERR_TIMEOUT in the status word, lets the copies land and returns, leaving the context
 * usable after guard_reset.  Exists so that the bounded-wait path can be exercised. */
int guard_debug_set_wait_limit(guard_ctx *ctx, long long cycles);

/* Synchronises `stream` and returns the sticky device status of the context
 * (GUARD_OK, GUARD_ERR_NONFINITE, GUARD_ERR_TIMEOUT, GUARD_ERR_INTERNAL, GUARD_ERR_CUDA). */
int guard_sync_status(guard_ctx *ctx, void *stream);

/* Clears the ring position, exceedance ring, consecutive counters and status. */
int guard_reset(guard_ctx *ctx, void *stream);

/* Enables (default) or disables the internal fork/join stream described under Conventions. */
int guard_set_overlap(guard_ctx *ctx, int on);

/* Sliding evaluations (on by default).  When an evaluation follows the previous one by at most 8
 * steps (the online monitor of Sec. 4.2 / 7.1 re-evaluates every step or poll), consecutive
 * windows share almost all their steps; guard_score then updates a small per-series state (an
 * interval around the series' median, the count of window values below it, the values inside)
 * from the few steps that entered and left the window instead of reading the whole window again
 * (the steps that left must still be in the ring: capacity_steps >= W + the steps between two
 * evaluations, else every evaluation reads its whole window).
 * Series whose median has left their interval are rebuilt from the window.  Results are identical
 * either way; guard_set_sliding(ctx, 0) makes every evaluation read its whole window. */
int guard_set_sliding(guard_ctx *ctx, int on);

/* Single rows of wide fleets (on by default).  The cross-rank statistics of a one-step ingest and
 * the fleet baseline of an evaluation (Sec. 4.2: median and MAD over all ranks) are each ONE row; from
 * 8 192 ranks on, a call site keeps its previous median and MAD and a tuned width per metric, which
 * bracket the next row's: the selection then counts the values below the bracket, bins the few inside
 * and ranks the wanted bin's values directly.  The counts prove the bracket; a row they do not prove
 * (the first one, a jump, ties) takes the general selection inside the same kernel.  Blocks of many
 * steps (4 096 ranks and more, 4 or 8 metrics) use the same idea: the medians and MADs a block found
 * stay in its scratch and bracket those of the next block at the same step position, so nothing is
 * sampled; a step whose counts do not prove its bracket is redone exactly (it counts in
 * guard_fallback_steps) and samples next time.  Results are identical either way;
 * guard_set_row_hints(ctx, 0) always takes the general selection / sampled intervals. */
int guard_set_row_hints(guard_ctx *ctx, int on);

/* Diagnostic: synchronises `stream` and fills out[6] (HOST): single rows seen and (row, metric)
 * columns whose median and MAD both came out of their brackets, 0-1 for ingested steps, 2-3 for
 * fleet baselines (zero where hints do not apply); 4-5: evaluations whose top-k list (Sec. 4.2: the
 * slowest ranks) came from the candidates above the previous evaluation's threshold, and
 * evaluations that had to rank all ranks instead (evaluations at most 8 steps apart try the
 * threshold first; the list is identical either way).  Since creation / reset / state import. */
int guard_row_hints(guard_ctx *ctx, uint32_t out[6], void *stream);

/* Deferred evaluations (off by default).  While on, guard_score enqueues the evaluation on
 * streams of the library's own, ordered after everything enqueued on `stream` so far, and
 * `stream` does NOT wait for it: the evaluation (Section 4.2's peer comparison over the last
 * window) then runs beside the next guard_ingest instead of in front of it.  The output
 * buffers of that guard_score call are complete, in the order of a stream, only after that
 * stream has passed the next guard_score, guard_join, guard_sync_status or guard_reset on
 * this context; until then the caller must neither read nor reuse them.  At most one
 * evaluation is pending.  In this mode guard_ingest, too, may run its kernels on streams of the
 * library's own (two, taken in turn, ordered after everything enqueued on `stream` so far) when
 * the caller passes no d_step_med / d_step_mad: consecutive blocks then overlap one another;
 * the same calls as above make `stream` wait for them.  The ring slots of the pending evaluation's window must not be
 * overwritten, nor those of blocks whose kernels still run: guard_ingest waits by itself when its block reuses them,
 * and guard_ring_reserve refuses (GUARD_ERR_NOT_READY) to hand them out, since it cannot
 * order the caller's writes; with capacity_steps >= W + block size neither ever happens.
 * Results are identical to the default mode. */
int guard_set_deferred(guard_ctx *ctx, int on);

/* Makes `stream` wait for the pending deferred evaluation, if there is one (no host
 * synchronisation). */
int guard_join(guard_ctx *ctx, void *stream);

/* Kernel timing for benchmarks.  on = 1: guard_ingest records a pair of CUDA events on its
 * stream right around the longest of its kernels (the MAD / exceedance sweep of the split
 * cross-rank path; contexts whose sizes take another path record around their main kernel or
 * nothing).  on = 2: guard_score records the pair around its window-median kernel, on the
 * stream that kernel runs on.  guard_profile_read waits for the recorded events, returns the
 * sum of the kernel durations in milliseconds and their number, and forgets them.  on = 0
 * (default) switches it off and destroys any events not yet read; do not leave it on in a
 * long-running service without reading (events accumulate in host memory). */
int guard_profile_enable(guard_ctx *ctx, int on);
int guard_profile_read(guard_ctx *ctx, double *total_ms, int64_t *launches);

/* Steps ingested since creation or the last reset. */
int64_t guard_steps_seen(const guard_ctx *ctx);

/* Kernels this context has enqueued so far (host-side count; copies and memsets are not
 * counted). */
int64_t guard_kernel_launches(const guard_ctx *ctx);

/* Synchronises `stream` and returns how many cross-rank rows (ingested steps or fleet
 * baselines) had to be recomputed by the slower direct selection since creation or the last
 * reset, because the sampled interval of the fast path did not hold the middle elements or a
 * candidate list overflowed.  Results are exact either way; this is a performance counter.
 * Negative on error. */
int64_t guard_fallback_steps(guard_ctx *ctx, void *stream);

/* Diagnostic companion of guard_fallback_steps: synchronises `stream` and fills out[6] (HOST)
 * with event counts since creation / reset: 0 a CTA's staged candidate list overflowed, 1 a
 * step's candidate list overflowed, 2 the deferred-exceedance list overflowed, 3 the sampled
 * interval missed the median, 4 candidate selection inconsistent, 5 the interval missed the MAD. */
int guard_fallback_reasons(guard_ctx *ctx, uint32_t out[6], void *stream);

/* Diagnostic: synchronises `stream` and fills out[6] (HOST) with counts, since creation / reset,
 * of the series whose windowed median the one-thread-per-series kernel handed to its whole-warp
 * fallback: 0 in total, 1 no usable search interval, 2 more values inside the interval than it
 * keeps, 3 the median lay below the interval, 4 above it, 5 the selection did not converge.
 * Results are exact either way. */
int guard_window_fallbacks(guard_ctx *ctx, uint32_t out[6], void *stream);

/* Diagnostic: synchronises `stream` and returns how many series the sliding evaluations
 * (guard_set_sliding) rebuilt from their whole window since creation / reset (every series once
 * when sliding starts, afterwards those whose median left its interval).  Negative on error. */
int64_t guard_sliding_rebuilds(guard_ctx *ctx, void *stream);

/* Frees the host object (the workspace stays the caller's). NULL is allowed. */
void guard_destroy(guard_ctx *ctx);

/* Text of the last host-side error of this context (or of the last failed
 * guard_create / guard_sweep_qualify when ctx is NULL).  Never NULL. */
const char *guard_last_error(const guard_ctx *ctx);

/* Host helper: the order-preserving float32 -> uint32 key the kernels select on
 * (total order of finite floats equals unsigned order of keys), and its inverse. */
uint32_t guard_key_from_float(float x);
float guard_float_from_key(uint32_t key);

#ifdef __cplusplus
}
#endif
#endif /* GUARD_B200_H */
