// Fused evaluation pass: k-of-W exceedance counts, robust deviation score, per-metric
// threshold and persistence, the multi-signal flag with the step-time metric as primary
// signal, the response tier and the consecutive-evaluation counter -- one thread per rank.
#include "kernels.h"

namespace guard {

namespace {

constexpr int kScoreThreads = 128;

// Scores of the ranks a top-k selection has already picked (first CTA only): the same float32
// arithmetic as the per-rank scores.
__device__ __forceinline__ void topk_scores(const ScoreArgs &a, const MetricParams &p, const float *s_B, const float *s_Ds) {
    if (blockIdx.x != 0 || !a.topk_score || !a.topk_idx) return;
    const int pm = p.primary;
    for (int i = threadIdx.x; i < a.K; i += blockDim.x) {
        const int r = a.topk_idx[i];
        float dev = __fsub_rn(a.wmed[(size_t)r * a.M + pm], s_B[pm]);
        if (p.dir[pm] < 0) dev = -dev;
        a.topk_score[i] = (dev == 0.0f) ? 0.0f : __fdiv_rn(__fmul_rn(0.6745f, dev), s_Ds[pm]);
    }
}

template <typename MaskT, int NM>
__global__ void __launch_bounds__(kScoreThreads) score_flag_kernel(const ScoreArgs a, const MetricParams p) {
    __shared__ float s_B[kMaxMetrics], s_rhs[kMaxMetrics], s_Ds[kMaxMetrics];
    const int M = a.M;
    if (threadIdx.x < M) {
        const int m = threadIdx.x;
        const float B = a.fleet_med[m];
        const float Ds = scale_of(a.fleet_mad[m], B, p.floor_rel[m], p.floor_abs[m]);
        s_B[m] = B;
        s_Ds[m] = Ds;
        s_rhs[m] = __fmul_rn(p.thrp[m], Ds);
    }
    __syncthreads();
    topk_scores(a, p, s_B, s_Ds);
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= a.R) return;

    // persistence: recount this rank's exceedance bits over the window's steps
    int cnt[NM];
#pragma unroll
    for (int m = 0; m < NM; ++m) cnt[m] = 0;
    const MaskT *mask_base = (const MaskT *)a.mask_base;
    int slot = ((a.last_slot - (a.n - 1)) % a.capacity + a.capacity) % a.capacity;
    if (a.slide) {
        // the previous window's counts, minus the steps that left, plus the steps that entered
#pragma unroll
        for (int m = 0; m < NM; ++m)
            if (m < M) cnt[m] = a.kcnt[(size_t)r * M + m];
        for (int i = 0; i < a.leaving; ++i) {
            int sl = slot - a.leaving + i;
            if (sl < 0) sl += a.capacity;
            const uint32_t e = mask_base[(size_t)sl * a.R + r];
#pragma unroll
            for (int m = 0; m < NM; ++m) cnt[m] -= (e >> m) & 1u;
        }
        for (int i = 0; i < a.entering; ++i) {
            int sl = a.last_slot - i;
            if (sl < 0) sl += a.capacity;
            const uint32_t e = mask_base[(size_t)sl * a.R + r];
#pragma unroll
            for (int m = 0; m < NM; ++m) cnt[m] += (e >> m) & 1u;
        }
    } else {
        for (int j = 0; j < a.n; ++j) {
            const uint32_t e = mask_base[(size_t)slot * a.R + r];
#pragma unroll
            for (int m = 0; m < NM; ++m) cnt[m] += (e >> m) & 1u;
            if (++slot == a.capacity) slot = 0;
        }
    }
    if (a.kcnt) {
#pragma unroll
        for (int m = 0; m < NM; ++m)
            if (m < M) a.kcnt[(size_t)r * M + m] = (uint16_t)cnt[m];
    }

    uint32_t mask = 0;
    const float *w = a.wmed + (size_t)r * M;
#pragma unroll
    for (int m = 0; m < NM; ++m) {
        if (m < M) {
            const float x = w[m];
            float dev = __fsub_rn(x, s_B[m]);
            if (p.dir[m] < 0) dev = -dev;
            const bool zflag = dev > s_rhs[m];
            if (zflag && cnt[m] >= p.k) mask |= 1u << m;
            if (a.counts) a.counts[(size_t)r * M + m] = (uint16_t)cnt[m];
            if (a.scores) a.scores[(size_t)r * M + m] = (dev == 0.0f) ? 0.0f : __fdiv_rn(__fmul_rn(0.6745f, dev), s_Ds[m]);
        }
    }
    const int need = min(p.min_signals, M);
    const bool cand = ((mask >> p.primary) & 1u) && (__popc(mask) >= need);
    int c = a.consec[r];
    c = cand ? min(c + 1, 255) : 0;
    a.consec[r] = (uint8_t)c;
    const bool flag = cand && (c >= p.n_consec);
    const int pm = p.primary;
    float devp = __fsub_rn(w[pm], s_B[pm]);
    if (p.dir[pm] < 0) devp = -devp;
    const float absB = fabsf(s_B[pm]);
    int t = 0;
    if (flag && devp >= __fmul_rn(p.tier_severe, absB)) t = 3;
    else if (flag && devp >= __fmul_rn(p.tier_moderate, absB)) t = 2;
    else if (mask != 0) t = 1;
    if (a.metric_mask) a.metric_mask[r] = mask;
    if (a.flags) a.flags[r] = (uint8_t)flag;
    if (a.tier) a.tier[r] = (uint8_t)t;
    a.flags_keep[r] = (uint8_t)flag;
    a.tier_keep[r] = (uint8_t)t;
}


// Byte-wide exceedance masks (at most 8 metrics): a CTA scores 128 ranks.  The recount over
// the window is split over the CTA's eight warps (warp w takes steps w, w + 8, ...); every
// thread loads the mask bytes of four adjacent ranks as one 32-bit word and accumulates
// metric m of all four in the byte lanes of one register ((word >> m) & 0x01010101), so a
// window step costs one coalesced 128-byte load per warp.  Partial counts meet in shared
// memory, then one thread per rank does the scoring.
constexpr int kFastRanks = 128;
constexpr int kFastWarps = 8;

__global__ void __launch_bounds__(kFastWarps * 32) score_flag_bytes_kernel(const ScoreArgs a, const MetricParams p) {
    __shared__ float s_B[8], s_rhs[8], s_Ds[8];
    const int M = a.M, tid = threadIdx.x, lane = lane_id(), w = warp_id();
    if (tid < M) {
        const float B = a.fleet_med[tid];
        const float Ds = scale_of(a.fleet_mad[tid], B, p.floor_rel[tid], p.floor_abs[tid]);
        s_B[tid] = B;
        s_Ds[tid] = Ds;
        s_rhs[tid] = __fmul_rn(p.thrp[tid], Ds);
    }
    __syncthreads();
    topk_scores(a, p, s_B, s_Ds);
    const int r0 = blockIdx.x * kFastRanks;
    const uint8_t *mask_base = (const uint8_t *)a.mask_base;
    const int first = ((a.last_slot - (a.n - 1)) % a.capacity + a.capacity) % a.capacity;
    const int rq = r0 + 4 * lane;                 // this lane's four ranks
    const bool word_ok = (rq + 3 < a.R) && ((a.R & 3) == 0);
    uint32_t acc[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) acc[m] = 0;
    uint32_t sums[4][8];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int m = 0; m < 8; ++m) sums[q][m] = 0;
    int pending = 0;
    constexpr int KU = 5;   // window steps whose loads are in flight together
    for (int j0 = w; !a.slide && j0 < a.n; j0 += kFastWarps * KU) {
        uint32_t word[KU];
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            const int j = j0 + u * kFastWarps;
            word[u] = 0;
            if (j < a.n) {
                int slot = first + j;
                if (slot >= a.capacity) slot -= a.capacity;
                const uint8_t *rowp = mask_base + (size_t)slot * a.R;
                if (word_ok) {
                    word[u] = __ldg(reinterpret_cast<const uint32_t *>(rowp + rq));
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (rq + q < a.R) word[u] |= (uint32_t)rowp[rq + q] << (8 * q);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < KU; ++u)
#pragma unroll
            for (int m = 0; m < 8; ++m) acc[m] += (word[u] >> m) & 0x01010101u;
        pending += KU;
        if (pending > 255 - KU) {   // byte lanes are about to overflow: spill into the wide sums
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int m = 0; m < 8; ++m) sums[q][m] += (acc[m] >> (8 * q)) & 255u;
#pragma unroll
            for (int m = 0; m < 8; ++m) acc[m] = 0;
            pending = 0;
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int m = 0; m < 8; ++m) sums[q][m] += (acc[m] >> (8 * q)) & 255u;
    // the eight warps' partial counts meet in shared memory
    __shared__ uint32_t s_cnt[kFastRanks][8];
    for (int i = tid; i < kFastRanks * 8; i += blockDim.x) (&s_cnt[0][0])[i] = 0;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int m = 0; m < 8; ++m)
            if (sums[q][m]) atomicAdd(&s_cnt[4 * lane + q][m], sums[q][m]);
    __syncthreads();
    if (tid >= kFastRanks) return;
    const int r = r0 + tid;
    if (r >= a.R) return;
    // sliding counts: the exceedance bytes of the few steps that left and entered the window, for this rank
    int slide_delta[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (a.slide) {
        for (int i = 0; i < a.leaving; ++i) {
            int sl = first - a.leaving + i;
            if (sl < 0) sl += a.capacity;
            const uint32_t e = mask_base[(size_t)sl * a.R + r];
#pragma unroll
            for (int m = 0; m < 8; ++m) slide_delta[m] -= (int)((e >> m) & 1u);
        }
        for (int i = 0; i < a.entering; ++i) {
            int sl = a.last_slot - i;
            if (sl < 0) sl += a.capacity;
            const uint32_t e = mask_base[(size_t)sl * a.R + r];
#pragma unroll
            for (int m = 0; m < 8; ++m) slide_delta[m] += (int)((e >> m) & 1u);
        }
    }
    uint32_t mask = 0;
    const float *wv = a.wmed + (size_t)r * M;
#pragma unroll
    for (int m = 0; m < 8; ++m) {
        if (m < M) {
            int cnt = (int)s_cnt[tid][m];
            if (a.slide) cnt = (int)a.kcnt[(size_t)r * M + m] + slide_delta[m];
            if (a.kcnt) a.kcnt[(size_t)r * M + m] = (uint16_t)cnt;
            float dev = __fsub_rn(wv[m], s_B[m]);
            if (p.dir[m] < 0) dev = -dev;
            if (dev > s_rhs[m] && cnt >= p.k) mask |= 1u << m;
            if (a.counts) a.counts[(size_t)r * M + m] = (uint16_t)cnt;
            if (a.scores) a.scores[(size_t)r * M + m] = (dev == 0.0f) ? 0.0f : __fdiv_rn(__fmul_rn(0.6745f, dev), s_Ds[m]);
        }
    }
    const int need = min(p.min_signals, M);
    const bool cand = ((mask >> p.primary) & 1u) && (__popc(mask) >= need);
    int c = a.consec[r];
    c = cand ? min(c + 1, 255) : 0;
    a.consec[r] = (uint8_t)c;
    const bool flag = cand && (c >= p.n_consec);
    const int pm = p.primary;
    float devp = __fsub_rn(wv[pm], s_B[pm]);
    if (p.dir[pm] < 0) devp = -devp;
    const float absB = fabsf(s_B[pm]);
    int t = 0;
    if (flag && devp >= __fmul_rn(p.tier_severe, absB)) t = 3;
    else if (flag && devp >= __fmul_rn(p.tier_moderate, absB)) t = 2;
    else if (mask != 0) t = 1;
    if (a.metric_mask) a.metric_mask[r] = mask;
    if (a.flags) a.flags[r] = (uint8_t)flag;
    if (a.tier) a.tier[r] = (uint8_t)t;
    a.flags_keep[r] = (uint8_t)flag;
    a.tier_keep[r] = (uint8_t)t;
}

// Node-level fold.  A CTA takes 32 nodes; its eight warps split the window's steps (warp w takes
// steps w, w + 8, ...), lane l owns node l of the CTA's 32.  "All ranks of the node exceeded on the
// primary metric in this step" is an AND over the node's exceedance entries; with eight ranks per
// node and byte-wide entries that is one 64-bit load and one mask test.
constexpr int kNodeWarps = 8;

template <typename MaskT>
__global__ void __launch_bounds__(kNodeWarps * 32) node_verdict_kernel(const NodeArgs a) {
    __shared__ uint32_t s_stall[32];
    const int lane = lane_id(), w = warp_id();
    const int node = blockIdx.x * 32 + lane;
    if (threadIdx.x < 32) s_stall[threadIdx.x] = 0;
    __syncthreads();
    const bool live = node < a.nodes;
    const int rpn = a.ranks_per_node;
    const size_t r0 = (size_t)node * rpn;
    const MaskT *mask_base = (const MaskT *)a.mask_base;
    const int first = ((a.last_slot - (a.n - 1)) % a.capacity + a.capacity) % a.capacity;
    const bool wide = sizeof(MaskT) == 1 && rpn == 8 && (a.R & 7) == 0;
    const unsigned long long want = 0x0101010101010101ull << a.primary;
    uint32_t stall = 0;
    if (live) {
        for (int j = w; j < a.n; j += kNodeWarps) {
            int slot = first + j;
            if (slot >= a.capacity) slot -= a.capacity;
            const MaskT *rowp = mask_base + (size_t)slot * a.R + r0;
            bool all = true;
            if (wide) {
                all = (__ldg(reinterpret_cast<const unsigned long long *>(rowp)) & want) == want;
            } else {
                for (int q = 0; q < rpn; ++q) all = all && (((uint32_t)rowp[q] >> a.primary) & 1u);
            }
            stall += all;
        }
        if (stall) atomicAdd(&s_stall[lane], stall);
    }
    __syncthreads();
    if (w == 0 && live) {
        int any = 0, top = 0;
        for (int q = 0; q < rpn; ++q) {
            any |= a.flags[r0 + q];
            top = max(top, (int)a.tier[r0 + q]);
        }
        if (a.node_flag) a.node_flag[node] = (uint8_t)(any != 0);
        if (a.node_tier) a.node_tier[node] = (uint8_t)top;
        if (a.node_stall) a.node_stall[node] = (uint16_t)s_stall[lane];
    }
}

}  // namespace

cudaError_t launch_node_verdict(const NodeArgs &a, cudaStream_t st) {
    const int grid = (a.nodes + 31) / 32;
    if (a.mask_bytes == 1) node_verdict_kernel<uint8_t><<<grid, kNodeWarps * 32, 0, st>>>(a);
    else node_verdict_kernel<uint32_t><<<grid, kNodeWarps * 32, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_score_flag(const ScoreArgs &a, const MetricParams &p, cudaStream_t st) {
    const int grid = (a.R + kScoreThreads - 1) / kScoreThreads;
    if (a.mask_bytes == 1)
        score_flag_bytes_kernel<<<(a.R + kFastRanks - 1) / kFastRanks, kFastWarps * 32, 0, st>>>(a, p);
    else
        score_flag_kernel<uint32_t, 32><<<grid, kScoreThreads, 0, st>>>(a, p);
    return cudaGetLastError();
}

}  // namespace guard
