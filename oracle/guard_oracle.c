/*
 * guard_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded CPU statement of what the straggler-scoring path
 * computes, written from the definitions (full sort for every order statistic, full
 * recount for every window).  It exists so that the CUDA library can be checked
 * against it; it shares no code with that library and nothing in the product may
 * call it.  Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What the paper fixes (all in words, Section 4.2 "Online Monitoring Strategy" and
 * Sections 5.2-5.4 on the node sweep):
 *   - every metric is judged against the peers of the same job, never an absolute limit;
 *   - a rank is flagged only when several indicators deviate, and the deviation is
 *     sustained over evaluation windows, so that transient spikes do not flag;
 *   - training-step time is the primary signal, the other metrics support it;
 *   - response tiers: no visible impact ("pending verification"), a sustained
 *     slowdown of about 10 %, and a slowdown of 20 % or more;
 *   - a node returns to the pool only if every part of its sweep passes.
 * The paper names no statistic.  The statistics used here (median, median absolute
 * deviation, the 0.6745-scaled robust z with cut-off 3.5, k-of-W persistence, a
 * nearest-rank percentile) are readings of that wording; each function below says
 * which reading it implements.
 *
 * Arithmetic contract.  Inputs are finite float32.  Values are ordered by the IEEE
 * total order (so -0 sorts before +0).  Every decision (exceedance, flag, tier,
 * percentile cut, top-k order) uses only single float32 subtract, multiply, fabs and
 * compare, so that it is reproducible bit for bit; this file must be compiled with
 * -ffp-contract=off.  Reported robust-z scores are computed here in float64 from the
 * float32 statistics.
 *
 * Parity pins: tests/test_oracle_pins.py (hand examples, numpy's sort/median,
 * a pure-Python brute force, Gaussian closed form, invariants).  Detection quality
 * against the paper's false-positive / false-negative rates is "parity unpinned"
 * (it needs the production labels).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAX_METRICS 32
#define ROBUST_Z_CONST 0.6745 /* Phi^-1(3/4): MAD of a unit normal, to 4 digits */

typedef struct {
    int R, M, W, k, topk;
    int primary, min_signals, n_consec;
    float tier_moderate, tier_severe;
    int dir[ORACLE_MAX_METRICS];
    float thrp[ORACLE_MAX_METRICS]; /* (float)(thr / 0.6745) */
    float floor_rel[ORACLE_MAX_METRICS], floor_abs[ORACLE_MAX_METRICS];
    float *hist;         /* telemetry of the last W steps: hist[step % W][r][m] */
    unsigned char *exc;  /* per-step exceedance of the last W steps: exc[step % W][r][m] */
    long long seen;      /* steps ingested so far */
    unsigned char *consec; /* consecutive evaluations in which rank r was a candidate */
    unsigned char *last_flag, *last_tier; /* per-rank flag / tier of the last evaluation */
    long long eval_seen;   /* steps seen when that evaluation ran (-1: none yet) */
} oracle_t;

/* ---- order statistics -------------------------------------------------------------- */

/* IEEE total order on finite floats: numeric order, and -0 before +0. */
static int cmp_f32(const void *pa, const void *pb)
{
    float a = *(const float *)pa, b = *(const float *)pb;
    if (a < b) return -1;
    if (a > b) return 1;
    return (signbit(b) != 0) - (signbit(a) != 0);
}

/* Median by full sort.  Odd n: the middle element.  Even n: midpoint of the two
 * middle elements, one float32 add and one (exact) multiply by 0.5.  tmp has room
 * for n floats and returns sorted. */
static float median_sorted_copy(const float *v, long n, long stride, float *tmp)
{
    for (long i = 0; i < n; ++i) tmp[i] = v[i * stride];
    qsort(tmp, (size_t)n, sizeof(float), cmp_f32);
    if (n & 1) return tmp[(n - 1) / 2];
    return 0.5f * (tmp[n / 2 - 1] + tmp[n / 2]);
}

float oracle_median(const float *v, long n)
{
    float *tmp = (float *)malloc(sizeof(float) * (size_t)n);
    float m = median_sorted_copy(v, n, 1, tmp);
    free(tmp);
    return m;
}

/* Raw (unscaled) median absolute deviation about med: median_i |v_i - med|, the
 * difference taken in float32. */
static float mad_about(const float *v, long n, long stride, float med, float *tmp, float *tmp2)
{
    for (long i = 0; i < n; ++i) tmp2[i] = fabsf(v[i * stride] - med);
    return median_sorted_copy(tmp2, n, 1, tmp);
}

float oracle_mad(const float *v, long n, float med)
{
    float *tmp = (float *)malloc(sizeof(float) * (size_t)n);
    float *tmp2 = (float *)malloc(sizeof(float) * (size_t)n);
    float m = mad_about(v, n, 1, med, tmp, tmp2);
    free(tmp);
    free(tmp2);
    return m;
}

/* Spread used as the denominator of the robust z: the MAD, floored so that a
 * degenerate (constant or quantised) peer group does not divide by zero. */
static float scale_of(float mad, float med, float floor_rel, float floor_abs)
{
    float s = mad;
    float rel = floor_rel * fabsf(med);
    if (rel > s) s = rel;
    if (floor_abs > s) s = floor_abs;
    return s;
}

float oracle_scale(float mad, float med, float floor_rel, float floor_abs)
{
    return scale_of(mad, med, floor_rel, floor_abs);
}

/* Modified z-score cut-off moved to the right-hand side so that the test
 * 0.6745 * dev / scale > thr becomes dev > thrp * scale with no division. */
float oracle_thrp(float thr) { return (float)((double)thr / ROBUST_Z_CONST); }

/* One-sided peer-relative exceedance in the "worse" direction of the metric. */
static int exceeds(float x, float med, float scale, int dir, float thrp)
{
    float dev = x - med;
    if (dir < 0) dev = -dev;
    return dev > thrp * scale;
}

/* ---- online scoring ---------------------------------------------------------------- */

oracle_t *oracle_create(int R, int M, int W, int k, int topk, int primary, int min_signals, int n_consec,
                        float tier_moderate, float tier_severe, const signed char *dir, const float *thr,
                        const float *floor_rel, const float *floor_abs)
{
    if (R < 1 || M < 1 || M > ORACLE_MAX_METRICS || W < 1 || k < 1 || k > W || topk < 0 || topk > R ||
        primary < 0 || primary >= M)
        return NULL;
    oracle_t *o = (oracle_t *)calloc(1, sizeof(oracle_t));
    o->R = R; o->M = M; o->W = W; o->k = k; o->topk = topk;
    o->primary = primary; o->min_signals = min_signals; o->n_consec = n_consec;
    o->tier_moderate = tier_moderate; o->tier_severe = tier_severe;
    for (int m = 0; m < M; ++m) {
        o->dir[m] = dir[m] < 0 ? -1 : 1;
        o->thrp[m] = oracle_thrp(thr[m]);
        o->floor_rel[m] = floor_rel[m];
        o->floor_abs[m] = floor_abs[m];
    }
    o->hist = (float *)calloc((size_t)W * R * M, sizeof(float));
    o->exc = (unsigned char *)calloc((size_t)W * R * M, 1);
    o->consec = (unsigned char *)calloc((size_t)R, 1);
    o->last_flag = (unsigned char *)calloc((size_t)R, 1);
    o->last_tier = (unsigned char *)calloc((size_t)R, 1);
    o->eval_seen = -1;
    return o;
}

void oracle_destroy(oracle_t *o)
{
    if (!o) return;
    free(o->hist); free(o->exc); free(o->consec); free(o->last_flag); free(o->last_tier); free(o);
}

void oracle_reset(oracle_t *o)
{
    o->seen = 0;
    o->eval_seen = -1;
    memset(o->consec, 0, (size_t)o->R);
    memset(o->exc, 0, (size_t)o->W * o->R * o->M);
}

/* Ingest B steps of telemetry block[b][r][m].  For every step and metric: the
 * cross-rank median and MAD (the peer baseline of that step), then the per-rank
 * exceedance bit.  step_med / step_mad ([B][M]) may be NULL.  Returns -1 (and ingests
 * nothing) if any value is not finite. */
int oracle_ingest(oracle_t *o, const float *block, int B, float *step_med, float *step_mad)
{
    const int R = o->R, M = o->M;
    const long long total = (long long)B * R * M;
    for (long long i = 0; i < total; ++i)
        if (!isfinite(block[i])) return -1;
    float *tmp = (float *)malloc(sizeof(float) * (size_t)R);
    float *tmp2 = (float *)malloc(sizeof(float) * (size_t)R);
    for (int b = 0; b < B; ++b) {
        const float *row = block + (size_t)b * R * M;
        const long slot = (long)(o->seen % o->W);
        float *h = o->hist + (size_t)slot * R * M;
        unsigned char *e = o->exc + (size_t)slot * R * M;
        memcpy(h, row, sizeof(float) * (size_t)R * M);
        for (int m = 0; m < M; ++m) {
            float med = median_sorted_copy(row + m, R, M, tmp);
            float mad = mad_about(row + m, R, M, med, tmp, tmp2);
            float scale = scale_of(mad, med, o->floor_rel[m], o->floor_abs[m]);
            for (int r = 0; r < R; ++r)
                e[(size_t)r * M + m] = (unsigned char)exceeds(row[(size_t)r * M + m], med, scale, o->dir[m], o->thrp[m]);
            if (step_med) step_med[(size_t)b * M + m] = med;
            if (step_mad) step_mad[(size_t)b * M + m] = mad;
        }
        o->seen += 1;
    }
    free(tmp); free(tmp2);
    return 0;
}

/* Order used by the top-k list: larger "badness" key first, equal keys by lower rank.
 * Keys are compared in the total order. */
typedef struct { float key; int idx; } keyed_t;
static int cmp_keyed_desc(const void *pa, const void *pb)
{
    const keyed_t *a = (const keyed_t *)pa, *b = (const keyed_t *)pb;
    int c = cmp_f32(&a->key, &b->key);
    if (c) return -c;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

/* One evaluation over the window of the last n = min(W, seen) steps.
 * Outputs (any may be NULL): wmed[R][M], fleet_med[M], fleet_mad[M], scores[R][M]
 * (float64), counts[R][M], mask[R], flags[R], tier[R], topk_idx[topk], topk_score[topk]
 * (float64).  Updates the consecutive-evaluation counters.  Returns -2 before the
 * first step. */
int oracle_score(oracle_t *o, float *wmed_out, float *fleet_med, float *fleet_mad, double *scores,
                 uint16_t *counts, uint32_t *mask_out, unsigned char *flags, unsigned char *tier,
                 int32_t *topk_idx, double *topk_score)
{
    const int R = o->R, M = o->M, W = o->W;
    if (o->seen < 1) return -2;
    const long n = (long)(o->seen < W ? o->seen : W);
    float *wmed = (float *)malloc(sizeof(float) * (size_t)R * M);
    float *tmp = (float *)malloc(sizeof(float) * (size_t)(R > W ? R : W));
    float *tmp2 = (float *)malloc(sizeof(float) * (size_t)(R > W ? R : W));
    float *col = (float *)malloc(sizeof(float) * (size_t)W);
    float B[ORACLE_MAX_METRICS], D[ORACLE_MAX_METRICS], Ds[ORACLE_MAX_METRICS];

    /* windowed per-rank median: the rank's own typical value over the window, blind
     * to isolated spikes */
    for (int r = 0; r < R; ++r)
        for (int m = 0; m < M; ++m) {
            for (long j = 0; j < n; ++j) {
                long long step = o->seen - n + j;
                col[j] = o->hist[((size_t)(step % W) * R + r) * M + m];
            }
            wmed[(size_t)r * M + m] = median_sorted_copy(col, n, 1, tmp);
        }
    /* fleet baseline of the windowed medians */
    for (int m = 0; m < M; ++m) {
        B[m] = median_sorted_copy(wmed + m, R, M, tmp);
        D[m] = mad_about(wmed + m, R, M, B[m], tmp, tmp2);
        Ds[m] = scale_of(D[m], B[m], o->floor_rel[m], o->floor_abs[m]);
        if (fleet_med) fleet_med[m] = B[m];
        if (fleet_mad) fleet_mad[m] = D[m];
    }
    keyed_t *keys = (keyed_t *)malloc(sizeof(keyed_t) * (size_t)R);
    for (int r = 0; r < R; ++r) {
        uint32_t mask = 0;
        for (int m = 0; m < M; ++m) {
            float w = wmed[(size_t)r * M + m];
            /* k-of-W persistence: recount the stored per-step exceedances over the window */
            int cnt = 0;
            for (long j = 0; j < n; ++j) {
                long long step = o->seen - n + j;
                cnt += o->exc[((size_t)(step % W) * R + r) * M + m];
            }
            int zflag = exceeds(w, B[m], Ds[m], o->dir[m], o->thrp[m]);
            if (zflag && cnt >= o->k) mask |= (1u << m);
            if (counts) counts[(size_t)r * M + m] = (uint16_t)cnt;
            if (scores) {
                double dev = (double)o->dir[m] * ((double)w - (double)B[m]);
                scores[(size_t)r * M + m] = (dev == 0.0) ? 0.0 : ROBUST_Z_CONST * dev / (double)Ds[m];
            }
            if (wmed_out) wmed_out[(size_t)r * M + m] = w;
        }
        /* multi-signal rule with step time as the primary signal */
        int need = o->min_signals < M ? o->min_signals : M;
        int cand = ((mask >> o->primary) & 1u) && (__builtin_popcount(mask) >= need);
        int c = o->consec[r];
        c = cand ? (c < 255 ? c + 1 : 255) : 0;
        o->consec[r] = (unsigned char)c;
        int flag = (c >= o->n_consec) && cand;
        /* tier from the relative slowdown of the primary metric */
        const int p = o->primary;
        float devp = wmed[(size_t)r * M + p] - B[p];
        if (o->dir[p] < 0) devp = -devp;
        float absB = fabsf(B[p]);
        int t = 0;
        if (flag && devp >= o->tier_severe * absB) t = 3;
        else if (flag && devp >= o->tier_moderate * absB) t = 2;
        else if (mask != 0) t = 1;
        if (mask_out) mask_out[r] = mask;
        if (flags) flags[r] = (unsigned char)flag;
        if (tier) tier[r] = (unsigned char)t;
        o->last_flag[r] = (unsigned char)flag;
        o->last_tier[r] = (unsigned char)t;
        float key = wmed[(size_t)r * M + p];
        if (o->dir[p] < 0) key = -key;
        keys[r].key = key;
        keys[r].idx = r;
    }
    if (o->topk > 0 && (topk_idx || topk_score)) {
        qsort(keys, (size_t)R, sizeof(keyed_t), cmp_keyed_desc);
        const int p = o->primary;
        for (int i = 0; i < o->topk; ++i) {
            int r = keys[i].idx;
            if (topk_idx) topk_idx[i] = r;
            if (topk_score) {
                double dev = (double)o->dir[p] * ((double)wmed[(size_t)r * M + p] - (double)B[p]);
                topk_score[i] = (dev == 0.0) ? 0.0 : ROBUST_Z_CONST * dev / (double)Ds[p];
            }
        }
    }
    o->eval_seen = o->seen;
    free(keys); free(wmed); free(tmp); free(tmp2); free(col);
    return 0;
}

/* Node-level verdict of the last evaluation.  The paper acts on nodes, not on single
 * GPUs (Section 4.2: a flagged node leaves the pool; Section 7.1: 8 GPUs per node), so
 * the per-rank results are folded over each group of ranks_per_node consecutive ranks:
 *   node_flag[n]  = 1 when any rank of node n is flagged;
 *   node_tier[n]  = the highest response tier among its ranks (0 none, 1 pending
 *                   verification, 2 mitigate at the next checkpoint, 3 restart now);
 *   node_stall[n] = in how many steps of the evaluation's window EVERY rank of the node
 *                   exceeded the step's peer baseline on the primary metric at once
 *                   (a correlated whole-node stall, as opposed to one slow GPU).
 * Must follow oracle_score with no ingest in between; R must be a multiple of
 * ranks_per_node.  Returns -2 when there is no such evaluation, -1 on bad arguments.
 * Reading: the paper says only that the node is the unit; OR / max / all-ranks-at-once
 * are this file's reading of that. */
int oracle_node_verdict(oracle_t *o, int ranks_per_node, unsigned char *node_flag, unsigned char *node_tier,
                        uint16_t *node_stall)
{
    const int R = o->R, M = o->M, W = o->W;
    if (ranks_per_node < 1 || R % ranks_per_node != 0) return -1;
    if (o->eval_seen < 1 || o->eval_seen != o->seen) return -2;
    const long n = (long)(o->seen < W ? o->seen : W);
    const int nodes = R / ranks_per_node;
    for (int nd = 0; nd < nodes; ++nd) {
        int any = 0, top = 0;
        for (int q = 0; q < ranks_per_node; ++q) {
            const int r = nd * ranks_per_node + q;
            if (o->last_flag[r]) any = 1;
            if (o->last_tier[r] > top) top = o->last_tier[r];
        }
        int stall = 0;
        for (long j = 0; j < n; ++j) {
            long long step = o->seen - n + j;
            int all = 1;
            for (int q = 0; q < ranks_per_node; ++q) {
                const int r = nd * ranks_per_node + q;
                if (!o->exc[((size_t)(step % W) * R + r) * M + o->primary]) all = 0;
            }
            stall += all;
        }
        if (node_flag) node_flag[nd] = (unsigned char)any;
        if (node_tier) node_tier[nd] = (unsigned char)top;
        if (node_stall) node_stall[nd] = (uint16_t)stall;
    }
    return 0;
}

/* Repeat-offender rule of the triage workflow (Section 6): a node that enters triage
 * `limit` times within `period` (the paper: three times within a week) is marked for
 * termination instead of going through triage again.  times[0..n) are the entry times
 * of ONE node in seconds, non-decreasing.  terminate[i] = 1 when entry i is at least
 * the limit-th entry of the span [times[i] - period, times[i]] (both ends included:
 * "within a week" is read as at most one period apart). */
int oracle_triage(const int64_t *times, int n, int64_t period, int limit, unsigned char *terminate)
{
    if (n < 0 || period < 0 || limit < 1) return -1;
    for (int i = 0; i < n; ++i) {
        if (i > 0 && times[i] < times[i - 1]) return -1;
        int c = 0;
        for (int j = 0; j <= i; ++j)
            if (times[i] - times[j] <= period) ++c;
        terminate[i] = (unsigned char)(c >= limit);
    }
    return 0;
}

/* ---- offline node-sweep qualification ---------------------------------------------- */

/* S[g][rep][m], g = node * gpus_per_node + local gpu.  Per GPU and metric: the median
 * over the repetitions.  Per metric over the fleet: median, MAD, and the nearest-rank
 * percentile cut at the bad tail (pct_ppm parts per million).  A metric fails a GPU
 * when it is both a robust-z outlier in the bad direction and strictly inside the bad
 * tail; a GPU passes when no metric fails; a node passes when all its GPUs pass. */
int oracle_sweep(const float *S, int nodes, int gpus_per_node, int reps, int M, const signed char *dir,
                 const float *thr, const float *floor_rel, const float *floor_abs, int pct_ppm,
                 float *gpu_med, float *fleet_med, float *fleet_mad, float *fleet_cut, uint32_t *fail_mask,
                 unsigned char *gpu_pass, unsigned char *node_pass)
{
    const long G = (long)nodes * gpus_per_node;
    if (G < 1 || reps < 1 || M < 1 || M > ORACLE_MAX_METRICS || pct_ppm < 0 || pct_ppm > 1000000) return -1;
    for (long long i = 0; i < (long long)G * reps * M; ++i)
        if (!isfinite(S[i])) return -1;
    const long big = G > reps ? G : reps;
    float *tmp = (float *)malloc(sizeof(float) * (size_t)big);
    float *tmp2 = (float *)malloc(sizeof(float) * (size_t)big);
    float *gm = (float *)malloc(sizeof(float) * (size_t)G * M);
    uint32_t *fm = (uint32_t *)calloc((size_t)G, sizeof(uint32_t));
    for (long g = 0; g < G; ++g)
        for (int m = 0; m < M; ++m)
            gm[(size_t)g * M + m] = median_sorted_copy(S + (size_t)g * reps * M + m, reps, M, tmp);
    long long j = ((long long)pct_ppm * G + 999999) / 1000000; /* ceil(pct * G) */
    if (j < 1) j = 1;
    if (j > G) j = G;
    for (int m = 0; m < M; ++m) {
        float F = median_sorted_copy(gm + m, G, M, tmp);
        float Fm = mad_about(gm + m, G, M, F, tmp, tmp2);
        float Fs = scale_of(Fm, F, floor_rel[m], floor_abs[m]);
        float thrp = oracle_thrp(thr[m]);
        int d = dir[m] < 0 ? -1 : 1;
        (void)median_sorted_copy(gm + m, G, M, tmp); /* tmp = sorted ascending */
        float cut = d < 0 ? tmp[j - 1] : tmp[G - j];
        for (long g = 0; g < G; ++g) {
            float v = gm[(size_t)g * M + m];
            int zfail = exceeds(v, F, Fs, d, thrp);
            int pfail = d < 0 ? (v < cut) : (v > cut);
            if (zfail && pfail) fm[g] |= (1u << m);
        }
        if (fleet_med) fleet_med[m] = F;
        if (fleet_mad) fleet_mad[m] = Fm;
        if (fleet_cut) fleet_cut[m] = cut;
    }
    for (long g = 0; g < G; ++g) {
        if (fail_mask) fail_mask[g] = fm[g];
        if (gpu_pass) gpu_pass[g] = (unsigned char)(fm[g] == 0);
    }
    if (node_pass)
        for (int nd = 0; nd < nodes; ++nd) {
            int ok = 1;
            for (int q = 0; q < gpus_per_node; ++q) ok = ok && (fm[(size_t)nd * gpus_per_node + q] == 0);
            node_pass[nd] = (unsigned char)ok;
        }
    if (gpu_med) memcpy(gpu_med, gm, sizeof(float) * (size_t)G * M);
    free(tmp); free(tmp2); free(gm); free(fm);
    return 0;
}
