// Host-side launchers of the scoring kernels (internal to the library).
#pragma once
#include <utility>
#include <vector>

#include "common.cuh"

namespace guard {

// Cross-rank statistics of S rows of a [rows][R][M] float32 array.  Row s of the launch
// lives at base + ((first_slot + s) % capacity) * row_stride.
struct XrankArgs {
    const float *base;
    long long row_stride;   // floats between consecutive rows (R * M)
    int first_slot;
    int capacity;
    int R, M;
    float *med;             // [S][M] cross-rank median (never NULL)
    float *mad;             // [S][M] raw MAD about that median (never NULL)
    float *med_user;        // [S][M] copy for the caller, or NULL
    float *mad_user;        // [S][M] copy for the caller, or NULL
    float *cut;             // [S][M] extra order statistic (0-based rank cut_rank[m]), or NULL
    int cut_rank[kMaxMetrics];
    void *mask_base;        // exceedance mask rows [capacity][R] of mask_bytes each, or NULL
    int mask_bytes;         // 1 (M <= 8) or 4
    int check_finite;       // flag NaN / Inf in the status word
    uint32_t *status;
    uint32_t *only_flagged; // [S] or NULL: direct kernel processes step s only if nonzero, then clears it
    uint32_t *fallbacks;    // or NULL: counts the steps the direct kernel redid for the bracketed path
    void *hint;             // ColHintState of the call site (one row per call), or NULL: column kernels only
    uint32_t hint_epoch;    // split path: non-zero lets a block use the records the previous block left in its scratch
};

// Scratch of the bracketed path for up to S_max steps per launch.
struct XrankScratch {
    float *lo, *hi;          // [S_max][M] value interval holding the two middle elements
    float *dlo, *dhi;        // interval holding the MAD
    float *rhs_lo, *rhs_hi;  // range of the exceedance threshold over that interval
    uint32_t *cnt_lt;        // [S_max][M] elements below the interval
    uint32_t *ncand;         // [S_max][M] elements collected
    uint32_t *flag;          // [S_max] step must be redone by the direct path
    uint32_t *namb;          // [S_max] deferred exceedance decisions
    uint32_t *cand;          // [S_max][M][cap] float bits of the collected elements
    uint32_t *amb;           // [S_max][amb_cap] (rank << 5 | metric)
    uint32_t *reasons;       // [8] why steps left the fast path (diagnostic counters) or NULL
    int cap, amb_cap, S_max;
};
enum { kWhyCtaList = 0, kWhyStepList = 1, kWhyAmbList = 2, kWhyMedianMiss = 3, kWhySelect = 4, kWhyMadMiss = 5 };
// State a call site of the column kernels keeps between its rows (zero before first use): the previous
// median / MAD in the output arrays bracket the next ones; hw holds the tuned half-widths of the two
// brackets per metric (0: derive from the MAD; negative: rows left before the hint is tried again).
struct ColHintState {
    uint32_t rows;       // diagnostic: rows seen
    uint32_t settled;    // diagnostic: columns whose median and MAD both came out of their brackets
    uint32_t pad[2];
    uint32_t valid[kMaxMetrics];   // the output arrays hold a previous result of this call site for metric m
    float hw[2][kMaxMetrics];
    // every entry of metric m is written only by the leader of the cluster that handles column m, after all
    // CTAs of that cluster have read it: the CTAs of a cluster always decide alike
};
// One CTA per (row, metric) column with the column in registers: for a few rows at a time.
bool xrank_column_supported(int R);
cudaError_t launch_xrank_column(const XrankArgs &a, const MetricParams &p, int S, cudaStream_t st);
// One cluster of four CTAs per step (4 or 8 metrics, a few thousand ranks and more).
bool xrank_cluster_supported(int R, int M);
cudaError_t launch_xrank_cluster(const XrankArgs &a, const MetricParams &p, int S, uint32_t *reasons, cudaStream_t st,
                                 std::vector<std::pair<cudaEvent_t, cudaEvent_t>> *prof = nullptr);
// Six uniform kernels per block (sample, sweep, select, sweep, select, finish) with the kept
// elements in global scratch (4 or 8 metrics, a few thousand to ~20 000 ranks).
bool xrank_split_supported(int R, int M);
// Thread path of the window medians when consecutive windows share most of their steps (the median
// hardly moves): keys the interval is tuned to catch, weight of the newest median in its centre.
constexpr int kWindowNearTarget = 14;
constexpr float kWindowNearSmooth = 1.0f;
constexpr int kSplitMaxSteps = 256;   // steps per launch group of the split path (sizes its scratch)
size_t xrank_split_scratch_bytes(int R, int M, int S_max);
cudaError_t launch_xrank_split(const XrankArgs &a, const MetricParams &p, int S, void *scratch, uint32_t *reasons,
                               cudaStream_t st, std::vector<std::pair<cudaEvent_t, cudaEvent_t>> *prof = nullptr);
bool xrank_bracket_supported(int R, int M);
int xrank_scratch_steps(int R, int M, int want);
size_t xrank_scratch_small_bytes(int M, int S_max);   // must be zero before first use
size_t xrank_scratch_big_bytes(int R, int M, int S_max);
XrankScratch carve_xrank_scratch(void *small_base, void *big_base, int R, int M, int S_max);
cudaError_t launch_xrank_bracketed(const XrankArgs &a, const MetricParams &p, const XrankScratch &sc, int S,
                                   cudaStream_t st);

cudaError_t launch_xrank_direct(const XrankArgs &a, const MetricParams &p, int S, cudaStream_t st);

// Windowed per-series median over the last n ring rows ending at slot `last_slot`.
struct WindowArgs {
    const float *ring;
    long long row_stride;   // R * M
    int capacity;
    int last_slot;          // slot of the newest step
    int n;                  // window length in steps
    int series;             // R * M
    float *wmed;            // [series] (never NULL)
    const float *wmed_prev; // [series] the previous evaluation's medians (another buffer than wmed), or NULL
    int use_hint;           // wmed_prev holds the previous evaluation's medians: use them as first pivots
    float *wmed_user;       // or NULL
    float *spread;          // [series] tuned half-width of the thread path's interval (state), or NULL
    float *centre;          // [series] smoothed median: the centre of the thread path's interval (state), or NULL
    int target;             // number of keys the thread path's interval is tuned to catch (0: default)
    float smooth;           // weight of the newest median in the interval's centre (0: default)
    uint32_t *fb_list;      // [series] scratch: series the thread path leaves to its finishing kernel (why << 28 | series)
    uint32_t *fb_list_count;// [2] their number and the finishing kernel's ticket: zero before first use, self-resetting
    uint32_t *fb_count;     // [6] series the thread path's interval did not serve, in total and by reason (diagnostic), or NULL
    uint32_t *status;
    long long first_wait_cycles;   // limit of the warp path's wait for a staged tile (0: the default of about a second)
};
// Launches one kernel (thread, warp or staged path).
cudaError_t launch_window_select(const WindowArgs &a, cudaStream_t st);

// Sliding windows: per-series state that lets an evaluation which follows the previous one by a few
// steps read only the steps that entered and left the window.  A series keeps an interval [lo, hi]
// around its median, the number of window values below lo and the values inside the interval; the
// median is then a rank among those.  A series whose median leaves the interval (or whose interval
// overflows) rebuilds its state from the whole window.
constexpr int kIncSlots = 40;     // values a series' interval can hold
constexpr int kIncHalf = 8;      // ranks the interval reaches beyond the middle ranks when it is (re)built
constexpr int kIncMaxNew = 8;     // most steps between two evaluations the sliding update is used for
struct IncArgs {
    float *lo, *hi;               // [series] interval ends (inclusive)
    uint32_t *cnt;                // [series] bit 31: state valid; bits 16..23: values inside; bits 0..15: values below lo
    float *val;                   // [series][kIncSlots] the values inside the interval, ascending (total order)
    int rebuild_all;              // ignore the stored state: every series rebuilds
    int entering;                 // steps that entered the window since the state was current (the newest ones)
    int leaving;                  // steps that left it (those right before the window's oldest step)
    uint32_t *rebuilds;           // diagnostic counter or NULL
    uint32_t *rb_list;            // [series] scratch: the series this launch has to rebuild
    uint32_t *rb_count;           // [2] their number and the rebuild kernel's ticket: zero before first use, self-resetting
};
size_t window_inc_bytes(int series);   // per array: lo, hi, cnt take series * 4 bytes, val kIncSlots * series * 4
bool window_inc_supported(const WindowArgs &a);
cudaError_t launch_window_incremental(const WindowArgs &a, const IncArgs &inc, cudaStream_t st);
int window_launch_count(const WindowArgs &a);

// Fused k-of-W count, robust score, thresholds, multi-signal flag, tier, consecutive counter.
struct ScoreArgs {
    int R, M;
    const float *wmed;       // [R][M]
    const float *fleet_med;  // [M]
    const float *fleet_mad;  // [M]
    const void *mask_base;   // exceedance rows [capacity][R]
    int mask_bytes;
    int capacity;
    int last_slot;
    int n;                   // window length
    uint8_t *consec;         // [R] state
    float *scores;           // [R][M] or NULL
    uint16_t *counts;        // [R][M] or NULL
    uint32_t *metric_mask;   // [R] or NULL
    uint8_t *flags;          // [R] or NULL
    uint8_t *tier;           // [R] or NULL
    uint8_t *flags_keep;     // [R] the context's own copy (input of the node-level fold), never NULL
    uint8_t *tier_keep;      // [R] likewise
    // scores of an already selected top-k list (the selection itself needs no fleet statistics and runs
    // beside the fleet baseline): topk_score[i] = primary score of rank topk_idx[i]; NULL / 0 to skip
    const int32_t *topk_idx;
    float *topk_score;
    int K;
    // k-of-W counts kept across evaluations: kcnt [R][M] is rewritten by every evaluation; with slide != 0
    // it holds the counts of the previous evaluation's window and only the exceedance rows of the
    // `entering` newest steps and of the `leaving` steps right before the window's oldest step are read
    uint16_t *kcnt;
    int slide, entering, leaving;
};
cudaError_t launch_score_flag(const ScoreArgs &a, const MetricParams &p, cudaStream_t st);

// Node-level fold of an evaluation: any rank flagged, highest tier, and the number of window steps
// in which every rank of the node exceeded on the primary metric at once.
struct NodeArgs {
    int R, ranks_per_node, nodes, primary;
    const uint8_t *flags, *tier;   // [R] per-rank results of the evaluation
    const void *mask_base;         // exceedance rows [capacity][R]
    int mask_bytes, capacity, last_slot, n;
    uint8_t *node_flag;            // [nodes] or NULL
    uint8_t *node_tier;            // [nodes] or NULL
    uint16_t *node_stall;          // [nodes] or NULL
};
cudaError_t launch_node_verdict(const NodeArgs &a, cudaStream_t st);

// State the top-k of consecutive evaluations keeps (zero before first use): the threshold key the
// previous evaluation left (about three times K ranks lie at or above it), the list counter and
// ticket of the hinted pass, whether the full pass has to run, and diagnostic counters.
struct TopkHint {
    uint32_t valid, tau, count, ticket, need_full, hits, misses, pad;
};
// Block-then-grid top-k of dir * wmed[:, primary].
struct TopkArgs {
    int R, M, K;
    const float *wmed;
    const float *fleet_med;
    const float *fleet_mad;
    unsigned long long *cand;   // scratch [topk_blocks(R)][K]
    unsigned int *ticket;       // scratch, zero before first use (self-resetting)
    int32_t *idx;               // [K] or NULL
    int32_t *idx_keep;          // [K] second copy of the indices (the context's own), or NULL
    float *score;               // [K] or NULL: needs fleet_med / fleet_mad to be final when the kernel runs
    TopkHint *hint;             // or NULL: state of the hinted pass (evaluations a few steps apart; used when score is NULL)
    unsigned long long *hcand;  // scratch [1024] of the hinted pass
};
int topk_blocks(int R);
// Records the text guard_last_error(NULL) returns (defined next to the C ABI).
void set_global_error(const char *text);
cudaError_t launch_topk(const TopkArgs &a, const MetricParams &p, cudaStream_t st);

// Node sweep: per-GPU medians over repetitions, then the verdicts.
struct SweepMedArgs {
    const float *S;   // [G][reps][M]
    int G, reps, M;
    float *gmed;      // [G][M]
    float *gmed_user; // or NULL
    uint32_t *status; // or NULL
    uint32_t *list;        // [G * M] scratch: series the thread path leaves to its finishing kernel, or NULL (then the warp path runs)
    uint32_t *list_count;  // [1] their number (cleared by the launcher)
};
cudaError_t launch_sweep_medians(const SweepMedArgs &a, cudaStream_t st);

struct SweepVerdictArgs {
    int nodes, gpus_per_node, M;
    const float *gmed, *fleet_med, *fleet_mad, *fleet_cut;
    uint32_t *fail_mask;  // or NULL
    uint8_t *gpu_pass;    // or NULL
    uint8_t *node_pass;   // or NULL
};
cudaError_t launch_sweep_verdict(const SweepVerdictArgs &a, const MetricParams &p, cudaStream_t st);

}  // namespace guard
