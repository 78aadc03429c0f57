// Fused evaluation pass: k-of-W exceedance counts, robust deviation score, per-metric
// threshold and persistence, the multi-signal flag with the step-time metric as primary
// signal, the response tier and the consecutive-evaluation counter -- one thread per rank.
#include "kernels.h"

namespace guard {

namespace {

constexpr int kScoreThreads = 128;

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
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= a.R) return;

    // persistence: recount this rank's exceedance bits over the window's steps
    int cnt[NM];
#pragma unroll
    for (int m = 0; m < NM; ++m) cnt[m] = 0;
    const MaskT *mask_base = (const MaskT *)a.mask_base;
    int slot = ((a.last_slot - (a.n - 1)) % a.capacity + a.capacity) % a.capacity;
    for (int j = 0; j < a.n; ++j) {
        const uint32_t e = mask_base[(size_t)slot * a.R + r];
#pragma unroll
        for (int m = 0; m < NM; ++m) cnt[m] += (e >> m) & 1u;
        if (++slot == a.capacity) slot = 0;
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
}

}  // namespace

cudaError_t launch_score_flag(const ScoreArgs &a, const MetricParams &p, cudaStream_t st) {
    const int grid = (a.R + kScoreThreads - 1) / kScoreThreads;
    if (a.mask_bytes == 1)
        score_flag_kernel<uint8_t, 8><<<grid, kScoreThreads, 0, st>>>(a, p);
    else
        score_flag_kernel<uint32_t, 32><<<grid, kScoreThreads, 0, st>>>(a, p);
    return cudaGetLastError();
}

}  // namespace guard
