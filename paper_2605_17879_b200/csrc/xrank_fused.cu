// Cross-rank selection, fused path: a sample kernel plus ONE main launch, one CTA of 1024
// threads per step, for
// fleets whose candidate lists fit in shared memory (4 or 8 metrics, up to ~20 000 ranks
// with 8 metrics).  The step's row is streamed twice (the second time it comes out of L2):
//
//   0. sample      (a small kernel of its own, one 64-thread CTA per column) two warps sort 512
//                  strided samples each in registers; seven order statistics of the merged sample (middle +-
//                  delta, quartiles +- delta) give the interval [lo, hi] of the median and
//                  [dlo, dhi] of the MAD;
//   1. sweep       every element is counted if below lo and kept (shared-memory list) if
//                  inside [lo, hi];
//   2. select      per metric, a group of threads checks the counts and finds the exact
//                  middle elements among the kept ones (histogram over the interval on
//                  order-preserving keys, refined until a bin is a single key);
//   3. sweep       the same for |x - med| in [dlo, dhi]; exceedance bits are written for
//                  elements clear of the threshold's possible range, the others are deferred;
//   4. select      exact MAD, threshold, deferred elements settled.
//
// If an interval does not hold what it should (the counts tell) or a list overflows, the
// CTA recomputes its step with the direct radix select, so the result is exact either way.
#include "xrank_common.cuh"
#include "xrank_direct.cuh"

namespace guard {

namespace {

constexpr int kFuThreads = 1024;
constexpr int kFuRPT = 4;            // ranks per thread per sweep iteration
constexpr int kFuBins = 1024;        // histogram bins per metric group
constexpr int kFuAmb = 2048;         // deferred exceedance decisions per step
constexpr int kFuCandWords = 32768;  // kept elements, shared out over the metrics (128 KB)
constexpr int kFuSample = 1024;      // sampled ranks per column

__device__ __forceinline__ void group_bar(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

struct GroupSel {
    uint32_t warp_tot[8];
    uint32_t bin, before, cnt, vmin;
    int found;
};

// k-th smallest (0-based) of the union of two ascending arrays of n keys each.
__device__ __forceinline__ uint32_t kth_of_two(const uint32_t *A, const uint32_t *B, int n, int k) {
    int lo = max(0, k + 1 - n), hi = min(k + 1, n);
    while (lo < hi) {
        const int i = (lo + hi) >> 1, j = k + 1 - i;
        if (j > 0 && i < n && B[j - 1] > A[i]) lo = i + 1; else hi = i;
    }
    const int i = lo, j = k + 1 - lo;
    const uint32_t a = i > 0 ? A[i - 1] : 0u, b = j > 0 ? B[j - 1] : 0u;
    return max(a, b);
}

// Finds the bin of hist[kFuBins] holding 0-based rank k (the G threads of one group).
template <int G>
__device__ __forceinline__ void group_find_bin(const uint32_t *hist, GroupSel &gs, uint32_t k, int gt, int barid) {
    constexpr int BPT = kFuBins / G;
    const int lane = gt & 31, gw = gt >> 5;
    uint32_t loc[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) { loc[i] = hist[gt * BPT + i]; sum += loc[i]; }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
    if (lane == 31) gs.warp_tot[gw] = incl;
    if (gt == 0) gs.found = 0;
    group_bar(barid, G);
    uint32_t off = 0;
    for (int w = 0; w < gw; ++w) off += gs.warp_tot[w];
    const uint32_t excl = off + incl - sum;
    if (k >= excl && k < excl + sum) {
        uint32_t run = excl;
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            if (k >= run && k < run + loc[i]) { gs.bin = (uint32_t)(gt * BPT + i); gs.before = run; gs.cnt = loc[i]; gs.found = 1; }
            run += loc[i];
        }
    }
    group_bar(barid, G);
}

// Keys of ranks k and (if want_next) k + 1 among list[0..n) (raw float bits in shared
// memory), all of whose keys lie in [base, base + width].  Called by the G threads of a group.
template <int G>
__device__ bool group_select(const uint32_t *list, uint32_t n, uint32_t k, bool want_next, uint32_t base, uint32_t width,
                             uint32_t *hist, GroupSel &gs, int gt, int barid, uint32_t &v1, uint32_t &v2) {
    uint32_t krem = k, ceq = 0;
    bool ok = true;
    v1 = 0;
    for (;;) {
        const int bits = 32 - __clz(width);
        const int shv = bits > 10 ? bits - 10 : 0;
        for (int i = gt; i < kFuBins; i += G) hist[i] = 0;
        group_bar(barid, G);
        for (uint32_t i = gt; i < n; i += G) {
            const uint32_t off = key_of_bits(list[i]) - base;
            if (off <= width) atomicAdd(&hist[off >> shv], 1u);
        }
        group_bar(barid, G);
        group_find_bin<G>(hist, gs, krem, gt, barid);
        if (!gs.found) { ok = false; break; }
        krem -= gs.before;
        if (shv == 0) { v1 = base + gs.bin; ceq = gs.cnt; break; }
        base += gs.bin << shv;
        width = (1u << shv) - 1u;
        group_bar(barid, G);
    }
    v2 = v1;
    if (ok && want_next && krem + 1 >= ceq) {   // next order statistic: smallest key above v1
        if (gt == 0) gs.vmin = 0xFFFFFFFFu;
        group_bar(barid, G);
        uint32_t c = 0xFFFFFFFFu;
        for (uint32_t i = gt; i < n; i += G) {
            const uint32_t key = key_of_bits(list[i]);
            if (key > v1) c = min(c, key);
        }
        c = __reduce_min_sync(0xFFFFFFFFu, c);
        if ((gt & 31) == 0 && c != 0xFFFFFFFFu) atomicMin(&gs.vmin, c);
        group_bar(barid, G);
        v2 = gs.vmin;
        if (v2 == 0xFFFFFFFFu) ok = false;
    }
    group_bar(barid, G);
    return ok;
}

// Sample kernel of the fused path: one CTA of two warps per (step, metric) column.  Each warp
// sorts 512 strided samples of the column in registers; seven order statistics of the two
// merged halves (middle, middle +- delta, quartiles +- delta_q) go to scratch as keys.  It is a
// kernel of its own because the register sort wants more than the 64 registers a thread gets
// inside the 1024-thread fused kernel, and small CTAs spread evenly over the SMs.
__global__ void __launch_bounds__(64) xrank_sample_q_kernel(const XrankArgs a, const int delta, const int delta_q,
                                                            uint32_t *__restrict__ qout) {
    __shared__ uint32_t samp[2 * 512];
    const int m = blockIdx.x, t = blockIdx.y, tid = threadIdx.x, lane = lane_id(), h = warp_id();
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const int stride = R / kFuSample;
    uint32_t v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int e = h * 512 + lane * 16 + j;
        v[j] = f2key(__ldg(row + (size_t)(e * stride + (stride >> 1)) * M + m));
    }
    warp_bitonic_sort<16>(v, lane);
#pragma unroll
    for (int j = 0; j < 16; ++j) samp[h * 512 + lane * 16 + j] = v[j];
    __syncthreads();
    if (tid < 8) {
        const int qq = tid;
        const int mid = kFuSample / 2, q1 = kFuSample / 4, q3 = 3 * kFuSample / 4;
        int k = mid;
        if (qq == 0) k = mid - delta; else if (qq == 2) k = mid + delta;
        else if (qq == 3) k = q1 - delta_q; else if (qq == 4) k = q1 + delta_q;
        else if (qq == 5) k = q3 - delta_q; else if (qq == 6) k = q3 + delta_q;
        k = min(max(k, 0), kFuSample - 1);
        qout[((size_t)t * M + m) * 8 + qq] = kth_of_two(samp, samp + 512, 512, k);
    }
}

template <int NQ, typename MaskT>
__global__ void __launch_bounds__(kFuThreads, 1) xrank_fused_kernel(const XrankArgs a, const MetricParams p,
                                                                    const uint32_t *__restrict__ qin, uint32_t *reasons) {
    constexpr int M = 4 * NQ, G = kFuThreads / M, CAP = kFuCandWords / M, LPI = kFuThreads / NQ;
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t *cand = smem;                   // [M][CAP]; holds the sorted samples [M][2][512] during phase 0
    uint32_t *hist = smem + kFuCandWords;    // [M][kFuBins]; the direct path's histograms on fallback
    uint32_t *amb = hist + M * kFuBins;      // [kFuAmb]
    __shared__ GroupSel gsel[M];
    __shared__ XrShared xsh;
    __shared__ float s_lo[M], s_hi[M], s_dlo[M], s_dhi[M], s_med[M], s_rlo[M], s_rhi[M], s_rhs[M];
    __shared__ uint32_t s_q[M][8];
    __shared__ uint32_t s_cnt[M], s_ncand[M], s_namb;
    __shared__ int s_fail, s_shift[M];   // s_fail: 1 = interval missed somewhere (retry), 2 = give up

    const int t = blockIdx.x, tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    const int R = a.R;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const size_t so = (size_t)t * M;
    const int mg = tid / G, gt = tid % G, barid = 1 + mg;   // selection groups: one per metric
    const int q = tid & (NQ - 1), rl = tid / NQ;            // sweeps: quad of metrics, rank lane
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2), k2 = (uint32_t)(R / 2);

    if (tid < M) { s_cnt[tid] = 0; s_ncand[tid] = 0; }
    if (tid == 0) { s_namb = 0; s_fail = 0; }
    if (tid < M) s_shift[tid] = 0;

    // ---- 0. the sample kernel's order statistics -> intervals ---------------------------------
    if (tid < M * 8) s_q[tid >> 3][tid & 7] = qin[so * 8 + tid];
    __syncthreads();
    if (tid < M) {
        const int m = tid;
        s_lo[m] = key2f(s_q[m][0]);
        s_hi[m] = key2f(s_q[m][2]);
        // The MAD is the half-width d at which [med - d, med + d] holds half of the column.  The
        // span between the quartiles' outer (inner) sample neighbours holds more (less) than
        // half with high probability; for a column that is roughly symmetric about its median
        // the half-lengths of those spans bracket d.  (A miss is caught by the counts.)
        const float dlo = 0.5f * (key2f(s_q[m][5]) - key2f(s_q[m][4]));
        const float dhi = 0.5f * (key2f(s_q[m][6]) - key2f(s_q[m][3]));
        s_dlo[m] = dlo > 0.0f ? fdown(dlo) : 0.0f;
        s_dhi[m] = (dhi >= 0.0f && dhi < CUDART_INF_F) ? fup(dhi) : CUDART_INF_F;
    }
    __syncthreads();

    // ---- 1. median sweep -------------------------------------------------------------------
    for (int attempt = 0;; ++attempt) {
    {
        float lo[4], hi[4];
        int cnt[4] = {0, 0, 0, 0};
#pragma unroll
        for (int c = 0; c < 4; ++c) { lo[c] = s_lo[4 * q + c]; hi[c] = s_hi[4 * q + c]; }
        bool bad = false;
        for (int base = 0; base < R; base += LPI * kFuRPT) {
            float v[kFuRPT][4];
            uint32_t cm[4] = {0, 0, 0, 0};
#pragma unroll
            for (int j = 0; j < kFuRPT; ++j) {
                const int r = base + j * LPI + rl;
                float4 x = make_float4(CUDART_INF_F, CUDART_INF_F, CUDART_INF_F, CUDART_INF_F);
                if (r < R) x = __ldg(reinterpret_cast<const float4 *>(row + (size_t)r * M) + q);
                v[j][0] = x.x; v[j][1] = x.y; v[j][2] = x.z; v[j][3] = x.w;
            }
#pragma unroll
            for (int j = 0; j < kFuRPT; ++j) {
                const bool in = base + j * LPI + rl < R;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float x = v[j][c];
                    if (a.check_finite && in) bad |= nonfinite_bits(__float_as_uint(x));
                    cnt[c] += (x < lo[c]);
                    if (x >= lo[c] && x <= hi[c]) cm[c] |= 1u << j;
                }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int m = 4 * q + c;
                int excl, total;
                group_scan<NQ>(__popc(cm[c]), excl, total);
                uint32_t b0 = 0;
                if (lane == q && total) b0 = atomicAdd(&s_ncand[m], (uint32_t)total);
                uint32_t pos = __shfl_sync(0xFFFFFFFFu, b0, q) + excl;
#pragma unroll
                for (int j = 0; j < kFuRPT; ++j)
                    if ((cm[c] >> j) & 1u) {
                        if (pos < (uint32_t)CAP) cand[m * CAP + pos] = __float_as_uint(v[j][c]);
                        ++pos;
                    }
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int tot = group_sum<NQ>(cnt[c]);
            if (lane == q && tot) atomicAdd(&s_cnt[4 * q + c], (uint32_t)tot);
        }
        if (a.check_finite && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(a.status, kStatNonFinite);
    }
    __syncthreads();

    // ---- 2. median select ------------------------------------------------------------------
    {
        const int m = mg;
        const uint32_t clt = s_cnt[m], n = s_ncand[m];
        int why = -1, shift = 0;
        if (n > (uint32_t)CAP) why = kWhyCtaList;
        else if (clt > k1) { why = kWhyMedianMiss; shift = -1; }
        else if (k2 >= clt + n) { why = kWhyMedianMiss; shift = 1; }
        uint32_t v1 = 0, v2 = 0;
        if (why < 0) {
            const float flo = s_lo[m], fhi = s_hi[m];
            const uint32_t base = f2key(flo == 0.0f ? -0.0f : flo);
            const uint32_t width = f2key(fhi == 0.0f ? 0.0f : fhi) - base;
            if (!group_select<G>(cand + m * CAP, n, k1 - clt, even, base, width, hist + m * kFuBins, gsel[m], gt, barid, v1, v2))
                why = kWhySelect;
        }
        if (gt == 0) {
            if (why < 0) {
                const float med = median_from_keys(v1, v2, even);
                s_med[m] = med;
                a.med[so + m] = med;
                if (a.med_user) a.med_user[so + m] = med;
                const float rel = __fmul_rn(p.floor_rel[m], fabsf(med));
                s_rlo[m] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(s_dlo[m], rel), p.floor_abs[m]));
                s_rhi[m] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(s_dhi[m], rel), p.floor_abs[m]));
            } else {
                if (reasons) atomicAdd(reasons + why, 1u);
                s_shift[m] = shift;
                atomicMax(&s_fail, (shift != 0 && attempt == 0) ? 1 : 2);
            }
        }
    }
    __syncthreads();
    const int verdict = s_fail;
    __syncthreads();   // everyone has read the verdict before it is cleared for the next attempt
    if (verdict != 1) break;
    // The counts say on which side of its interval a column's middle lies: move that interval
    // by its own width (the kept-element lists cannot hold a wider one) and sweep once more.
    if (tid < M) {
        const float w = s_hi[tid] - s_lo[tid];
        if (s_shift[tid] < 0) { s_hi[tid] = s_lo[tid]; s_lo[tid] = s_lo[tid] - w; }
        if (s_shift[tid] > 0) { s_lo[tid] = s_hi[tid]; s_hi[tid] = s_hi[tid] + w; }
        s_shift[tid] = 0;
        s_cnt[tid] = 0;
        s_ncand[tid] = 0;
    }
    if (tid == 0) s_fail = 0;
    __syncthreads();
    }   // attempts of the median phase
    if (!s_fail) {
      for (int attempt = 0;; ++attempt) {
        if (tid < M) { s_cnt[tid] = 0; s_ncand[tid] = 0; }
        if (tid == 0) s_namb = 0;
        __syncthreads();

        // ---- 3. MAD + exceedance sweep ---------------------------------------------------
        float lo[4], hi[4], med[4], rlo[4], rhi[4];
        int dirv[4];
        int cnt[4] = {0, 0, 0, 0};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int m = 4 * q + c;
            lo[c] = s_dlo[m]; hi[c] = s_dhi[m]; med[c] = s_med[m]; rlo[c] = s_rlo[m]; rhi[c] = s_rhi[m];
            dirv[c] = p.dir[m];
        }
        for (int base = 0; base < R; base += LPI * kFuRPT) {
            float v[kFuRPT][4];
            uint32_t cm[4] = {0, 0, 0, 0};
#pragma unroll
            for (int j = 0; j < kFuRPT; ++j) {
                const int r = base + j * LPI + rl;
                float4 x = make_float4(CUDART_INF_F, CUDART_INF_F, CUDART_INF_F, CUDART_INF_F);
                if (r < R) x = __ldg(reinterpret_cast<const float4 *>(row + (size_t)r * M) + q);
                v[j][0] = x.x; v[j][1] = x.y; v[j][2] = x.z; v[j][3] = x.w;
            }
#pragma unroll
            for (int j = 0; j < kFuRPT; ++j) {
                const int r = base + j * LPI + rl;
                const bool in = r < R;
                uint32_t ebits = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float dev = __fsub_rn(v[j][c], med[c]);
                    const float d = in ? fabsf(dev) : CUDART_INF_F;
                    v[j][c] = d;
                    cnt[c] += (d < lo[c]);
                    if (d >= lo[c] && d <= hi[c]) cm[c] |= 1u << j;
                    const float sdev = dirv[c] < 0 ? -dev : dev;
                    if (in && sdev > rlo[c]) {
                        if (sdev > rhi[c]) {
                            ebits |= 1u << (4 * q + c);
                        } else {   // decided once the exact MAD is known
                            const uint32_t pos = atomicAdd(&s_namb, 1u);
                            if (pos < (uint32_t)kFuAmb) amb[pos] = ((uint32_t)r << 5) | (uint32_t)(4 * q + c);
                        }
                    }
                }
                if (a.mask_base) {
#pragma unroll
                    for (int d = 1; d < NQ; d <<= 1) ebits |= __shfl_xor_sync(0xFFFFFFFFu, ebits, d);
                    if (q == 0 && in) reinterpret_cast<MaskT *>(a.mask_base)[(size_t)slot * R + r] = (MaskT)ebits;
                }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int m = 4 * q + c;
                int excl, total;
                group_scan<NQ>(__popc(cm[c]), excl, total);
                uint32_t b0 = 0;
                if (lane == q && total) b0 = atomicAdd(&s_ncand[m], (uint32_t)total);
                uint32_t pos = __shfl_sync(0xFFFFFFFFu, b0, q) + excl;
#pragma unroll
                for (int j = 0; j < kFuRPT; ++j)
                    if ((cm[c] >> j) & 1u) {
                        if (pos < (uint32_t)CAP) cand[m * CAP + pos] = __float_as_uint(v[j][c]);
                        ++pos;
                    }
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int tot = group_sum<NQ>(cnt[c]);
            if (lane == q && tot) atomicAdd(&s_cnt[4 * q + c], (uint32_t)tot);
        }
        __syncthreads();

        // ---- 4. MAD select, threshold, deferred elements ------------------------------------
        {
            const int m = mg;
            const uint32_t clt = s_cnt[m], n = s_ncand[m];
            int why = -1, shift = 0;
            if (s_namb > (uint32_t)kFuAmb) why = kWhyAmbList;
            else if (n > (uint32_t)CAP) why = kWhyCtaList;
            else if (clt > k1) { why = kWhyMadMiss; shift = -1; }
            else if (k2 >= clt + n) { why = kWhyMadMiss; shift = 1; }
            uint32_t v1 = 0, v2 = 0;
            if (why < 0) {
                const uint32_t base = f2key(s_dlo[m]);
                const uint32_t width = f2key(s_dhi[m]) - base;
                if (!group_select<G>(cand + m * CAP, n, k1 - clt, even, base, width, hist + m * kFuBins, gsel[m], gt, barid, v1, v2))
                    why = kWhySelect;
            }
            if (gt == 0) {
                if (why < 0) {
                    const float mad = median_from_keys(v1, v2, even);
                    a.mad[so + m] = mad;
                    if (a.mad_user) a.mad_user[so + m] = mad;
                    s_rhs[m] = __fmul_rn(p.thrp[m], scale_of(mad, s_med[m], p.floor_rel[m], p.floor_abs[m]));
                } else {
                    if (reasons) atomicAdd(reasons + why, 1u);
                    s_shift[m] = shift;
                    atomicMax(&s_fail, (shift != 0 && attempt == 0) ? 1 : 2);
                }
            }
        }
        __syncthreads();
        const int verdict = s_fail;
        __syncthreads();
        if (verdict != 1) break;
        if (tid < M) {   // move the missed MAD intervals by their own width, as above
            const int m = tid;
            const float w = s_dhi[m] - s_dlo[m];
            if (s_shift[m] < 0) { s_dhi[m] = s_dlo[m]; s_dlo[m] = fmaxf(0.0f, s_dlo[m] - w); }
            if (s_shift[m] > 0) { s_dlo[m] = s_dhi[m]; s_dhi[m] = s_dhi[m] + w; }
            s_shift[m] = 0;
            const float rel = __fmul_rn(p.floor_rel[m], fabsf(s_med[m]));
            s_rlo[m] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(s_dlo[m], rel), p.floor_abs[m]));
            s_rhi[m] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(s_dhi[m], rel), p.floor_abs[m]));
        }
        if (tid == 0) s_fail = 0;
        __syncthreads();
      }   // attempts of the MAD phase
        if (!s_fail) {
            if (a.mask_base) {
                const uint32_t na = s_namb;
                for (uint32_t i = tid; i < na; i += kFuThreads) {
                    const uint32_t e = amb[i];
                    const uint32_t r = e >> 5, m = e & 31u;
                    if (exceeds(row[(size_t)r * M + m], s_med[m], p.dir[m], s_rhs[m])) {
                        const size_t idx = (size_t)slot * R + r;
                        if (sizeof(MaskT) == 1) {
                            unsigned int *w = reinterpret_cast<unsigned int *>(reinterpret_cast<uintptr_t>(a.mask_base) + (idx & ~(size_t)3));
                            atomicOr(w, (1u << m) << (8 * (idx & 3)));
                        } else {
                            atomicOr(reinterpret_cast<unsigned int *>(a.mask_base) + idx, 1u << m);
                        }
                    }
                }
            }
            return;
        }
    }
    // ---- fallback: the direct radix select recomputes the whole step ---------------------------
    __syncthreads();
    xrank_direct_step(a, p, t, hist, xsh);
    if (tid == 0 && a.fallbacks) atomicAdd(a.fallbacks, 1u);
}

}  // namespace

bool xrank_fused_supported(int R, int M) {
    if (M != 4 && M != 8) return false;
    if (R < 4 * kFuSample) return false;
    // kept fraction of a column: the sampled interval spans 2 * delta of kFuSample sample ranks
    // (median) and 4 * delta_q (MAD: one band around each quartile)
    const double sq = sqrt((double)kFuSample);
    const double frac_med = 2.0 * ceil(5.5 * 0.5 * sq) / kFuSample;
    const double frac_mad = 4.0 * ceil(0.5 * 4.0 * 0.612 * sq) / kFuSample;
    const double frac = frac_med > frac_mad ? frac_med : frac_mad;
    return frac * R * 1.15 <= (double)(kFuCandWords / M);
}

cudaError_t launch_xrank_fused(const XrankArgs &a, const MetricParams &p, int S, uint32_t *reasons, uint32_t *qscratch,
                               cudaStream_t st, std::vector<std::pair<cudaEvent_t, cudaEvent_t>> *prof) {
    if (S <= 0) return cudaSuccess;
    // half-widths in sample ranks: 5.5 standard deviations of the sampled median's rank; the
    // quartile intervals bracket a count, the sum of two quartile ranks (sd ~ 0.61 sqrt(s)), at
    // 4 standard deviations (a miss there costs one more sweep, not the direct path)
    const int delta = (int)ceil(5.5 * 0.5 * sqrt((double)kFuSample));
    const int delta_q = (int)ceil(0.5 * 4.0 * 0.612 * sqrt((double)kFuSample));
    const size_t smem = (size_t)(kFuCandWords + a.M * kFuBins + kFuAmb) * sizeof(uint32_t);
    const bool wide = a.mask_bytes == 4;
    xrank_sample_q_kernel<<<dim3(a.M, S), 64, 0, st>>>(a, delta, delta_q, qscratch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (prof) {
        if (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess) return cudaGetLastError();
        cudaEventRecord(ev0, st);
    }
    if (a.M == 8) {
        if (wide) {
            e = cudaFuncSetAttribute(xrank_fused_kernel<2, uint32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            xrank_fused_kernel<2, uint32_t><<<S, kFuThreads, smem, st>>>(a, p, qscratch, reasons);
        } else {
            e = cudaFuncSetAttribute(xrank_fused_kernel<2, uint8_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            xrank_fused_kernel<2, uint8_t><<<S, kFuThreads, smem, st>>>(a, p, qscratch, reasons);
        }
    } else {
        if (wide) {
            e = cudaFuncSetAttribute(xrank_fused_kernel<1, uint32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            xrank_fused_kernel<1, uint32_t><<<S, kFuThreads, smem, st>>>(a, p, qscratch, reasons);
        } else {
            e = cudaFuncSetAttribute(xrank_fused_kernel<1, uint8_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            xrank_fused_kernel<1, uint8_t><<<S, kFuThreads, smem, st>>>(a, p, qscratch, reasons);
        }
    }
    e = cudaGetLastError();
    if (prof) {
        cudaEventRecord(ev1, st);
        prof->emplace_back(ev0, ev1);
    }
    return e;
}

}  // namespace guard
