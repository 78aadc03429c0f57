// Cross-rank selection, split path: six uniform kernels per ingested block, for fleets of a
// few thousand to about sixteen thousand ranks with 4 or 8 metrics.  Every kernel does one kind
// of work on many small CTAs, so that the streaming sweeps run with all their warps streaming
// and the short, latency-bound selections of hundreds of columns overlap one another:
//
//   0. sample   one CTA per (step, four metrics): per metric 32 spread values are sorted in a
//               warp; their median and quartile span fix a linear map onto 2048 bins; about
//               4096 ranks of the step (runs of four, evenly spread) are counted into those bins;
//               the bins that hold the sample ranks middle +- delta and quartiles +- delta_q
//               give the interval [lo, hi] of the column's median and [dlo, dhi] of its MAD;
//   1. sweep    one CTA per (step, chunk of ranks): counts the elements below lo and keeps
//               those inside [lo, hi] -- first in a shared-memory list (one reservation per
//               warp and batch), copied to the step's list in global scratch at the end;
//   2. select   one CTA per column: proves from the counts that the interval holds the
//               middle ranks and finds them among the kept elements, held in registers, by
//               histogram refinement on order-preserving keys;
//   3. sweep    the same for |x - med| in [dlo, dhi]; elements that might exceed the
//               threshold are rare: those clear of the threshold's possible range set their
//               exceedance bit at once, the others are deferred to a per-step list;
//   4. select   exact MAD and threshold;
//   5. finish   one CTA per step settles the deferred elements -- or, if an interval missed,
//               a list overflowed or the sample was degenerate, recomputes the whole step
//               with the direct radix select, so the result is exact either way.
//
// The scratch (intervals, counters, kept lists: ~80 KB per step) stays in L2 between kernels.
#include <math_constants.h>

#include <mutex>

#include "xrank_common.cuh"
#include "xrank_direct.cuh"

namespace guard {

namespace {

constexpr int kSpThreads = 256;     // sweep CTA
constexpr int kSpU = 4;             // ranks per thread and sweep batch
constexpr int kSpSlice = 4096;      // ranks per sweep CTA
constexpr int kSpSlack = 128;       // words behind each shared-memory list that absorb the stores of a full list
constexpr int kSpAmb = 1024;        // deferred exceedance decisions per step
constexpr int kSpSample = 4096;     // target number of sampled ranks per column
constexpr int kSpSBins = 2048;      // sample histogram bins (16-bit counters, two per word)
constexpr int kSpBins = 1024;       // selection histogram bins
constexpr int kSpSelThreads = 128;  // sample / select CTA
constexpr int kSpJmax = 20;         // kept elements per thread the register selection can hold
constexpr int kSpJsmall = 12;       // ... and of its variant for short lists
constexpr int kSpSegs = 4;          // sweep CTAs per step the selection can gather from
constexpr int kSpMaxM = 8;
constexpr float kFltMax = 3.402823466e+38f;

struct SpGeom {
    int chunks;     // sweep CTAs per step
    int slice;      // ranks per sweep CTA (a multiple of 16)
    int cap;        // kept elements per metric and sweep CTA (its shared-memory list and its segment in global scratch)
    int stride;     // one run of four consecutive ranks is sampled out of every 4 * stride
    int s;          // number of sampled ranks
    int delta;      // half-width of the median interval in sample ranks
    int delta_q;    // half-width of the quartile intervals in sample ranks
};

// Per-column record in global scratch.
struct SpCol {
    float lo, hi, dlo, dhi;   // intervals of the median and of the MAD
    float med, rlo, rhi, rhs; // median; range of the exceedance threshold over [dlo, dhi]; exact threshold
    uint32_t cnt;             // elements below the current interval
    float mad;                // the column's MAD (kept for the next use of this record)
    uint32_t epoch;           // SpScratch::epoch of the launch that completed med / mad on the fast path (else 0)
    uint32_t pad;
};

struct SpScratch {
    SpCol *col;       // [S][M]
    uint32_t *fail;   // [S] the step goes to the direct path
    uint32_t *namb;   // [S] deferred exceedance decisions
    uint32_t *amb;    // [S][kSpAmb] (rank << 5 | metric)
    uint32_t *nseg;   // [S][M][chunks] kept elements of each sweep CTA
    uint32_t *list;   // [S][M][chunks][cap] kept elements (raw bits), one segment per sweep CTA
    uint32_t epoch;   // non-zero: records stamped with this value hold the previous results of the same step position
};

// ---- per-element operations of the sweeps, written out so that each is a fixed handful of
// instructions (compare, predicated add / predicated store) ---------------------------------
// cnt += !(x >= lo); packed += INC if lo <= x <= hi.
// Written without predicates (comparison results as 0 / -1 words): sixteen of these in a row
// would otherwise have the compiler shuffle predicates through registers.
template <uint32_t INC>
__device__ __forceinline__ void sp_cell_count(const float x, const float lo, const float hi, uint32_t &cnt, uint32_t &packed) {
    uint32_t ge, le;
    asm("set.ge.u32.f32 %0, %1, %2;" : "=r"(ge) : "f"(x), "f"(lo));
    asm("set.le.u32.f32 %0, %1, %2;" : "=r"(le) : "f"(x), "f"(hi));
    cnt += 1u + ge;               // + 1 unless x >= lo
    packed += (ge & le) & INC;
}
// if (lo <= x <= hi) { shared[addr] = x; addr += 4; }
__device__ __forceinline__ void sp_cell_keep(const float x, const float lo, const float hi, uint32_t &addr) {
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ge.f32 p, %1, %2;\n\tsetp.le.and.f32 q, %1, %3, p;\n\t@q st.shared.f32 [%0], %1;\n\t@q add.u32 %0, %0, 4;\n\t}"
                 : "+r"(addr)
                 : "f"(x), "f"(lo), "f"(hi)
                 : "memory");
}
// one step of an inclusive scan over lanes: incl += value of lane (lane - d) where that lane exists
__device__ __forceinline__ void sp_scan_step(uint32_t &incl, const int d) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 r;\n\tshfl.sync.up.b32 r|p, %0, %1, 0, 0xffffffff;\n\t@p add.u32 %0, %0, r;\n\t}"
                 : "+r"(incl)
                 : "r"(d));
}
__device__ __forceinline__ uint32_t sp_atoms_add(const uint32_t addr, const uint32_t v) {
    uint32_t old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}

// Ascending sort of one key per lane (bitonic network over shuffles).
__device__ __forceinline__ uint32_t sp_warp_sort(uint32_t x, const int lane) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1)
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, x, stride);
            const bool asc = (lane & size) == 0, upper = (lane & stride) != 0;
            x = (asc != upper) ? min(x, o) : max(x, o);
        }
    return x;
}

// ---- 0. sample ---------------------------------------------------------------------------------
struct SpSelShared {
    uint32_t hist[kSpBins];
    uint32_t warp_tot[kSpSelThreads / 32];
    uint32_t bin, before, cnt, vmin, scount, r1, r2;
    int found;
    uint32_t small[32];
};

constexpr int kSpSmpThreads = 256;                      // sample CTA: one per (step, quad of metrics)
constexpr int kSpSmpG = kSpSmpThreads / 4;              // threads per metric in the scan
constexpr int kSpSmpLoads = kSpSample / kSpSmpThreads;  // sampled ranks per thread

struct SpSampleShared {
    uint32_t hist[4][kSpBins];   // 2048 16-bit bins per metric
    uint32_t warp_tot[4][2];
    float inv_bw[4], off[4];
    int ok[4];
    uint32_t tk[6], tb[4][6];
};

// The sample of a step: runs of four consecutive ranks, one run every 4 * stride ranks, so
// that a warp's 128-bit loads use whole cache lines (a column-wise strided sample costs one
// line per value).  One CTA handles four metrics: every thread bins the four components of
// its float4 into the four histograms; then 64 threads per metric scan their histogram.
__global__ void __launch_bounds__(kSpSmpThreads, 3) xsplit_sample_kernel(const XrankArgs a, const SpGeom g, const SpScratch sc,
                                                                      uint32_t *reasons) {
    __shared__ SpSampleShared sh;
    const int q = blockIdx.x, t = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const int period = 4 * g.stride, first = (period - 4) >> 1;

    // The column records still hold what the previous block on this scratch found at the same step position:
    // consecutive blocks of a fleet have almost the same per-step cross-rank median and MAD, so those bracket
    // the new ones without sampling anything (five standard errors of the difference of two sample medians /
    // MADs of normal data to either side; a miss is caught by the counts and the step redone).  Anything
    // else (first use, a step that left the fast path, a zero MAD) samples.
    __shared__ int s_hinted[4];
    if (tid < 4) {
        const SpCol &old = sc.col[(size_t)t * M + 4 * q + tid];
        const float om = old.med, od = old.mad;
        const bool v = sc.epoch != 0u && old.epoch == sc.epoch && od > 0.0f && od < kFltMax && fabsf(om) < kFltMax;
        s_hinted[tid] = v ? 1 : 0;
    }
    __syncthreads();
    if (s_hinted[0] && s_hinted[1] && s_hinted[2] && s_hinted[3]) {
        if (tid < 4) {
            SpCol &col = sc.col[(size_t)t * M + 4 * q + tid];
            const float om = col.med, od = col.mad;
            const float u = od * rsqrtf((float)R);
            const float hm = 13.1f * u, hd = 8.25f * u;
            col.lo = fmaxf(om - hm, -kFltMax);
            col.hi = fminf(om + hm, kFltMax);
            col.dlo = fmaxf(od - hd, 0.0f);
            col.dhi = fminf(od + hd, kFltMax);
            col.cnt = 0;
            col.epoch = 0;   // stamped again when this block's median and MAD are complete
        }
        if (tid == 0 && q == 0) { sc.fail[t] = 0; sc.namb[t] = 0; }
        return;
    }

    // all loads first: the sampled ranks, and (warps 0..3) the 32 spread values that fix a metric's bin map
    float4 xs[kSpSmpLoads];
#pragma unroll
    for (int j = 0; j < kSpSmpLoads; ++j) {
        const int i = tid + j * kSpSmpThreads;   // index into the sample
        xs[j] = make_float4(CUDART_NAN_F, CUDART_NAN_F, CUDART_NAN_F, CUDART_NAN_F);
        if (i < g.s) xs[j] = __ldg(reinterpret_cast<const float4 *>(row + (size_t)((i >> 2) * period + first + (i & 3)) * M) + q);
    }
    float xpre = 0.0f;
    if (warp < 4) xpre = __ldg(row + (size_t)min(R - 1, (int)(((long long)(2 * lane + 1) * R) >> 6)) * M + 4 * q + warp);
    for (int i = tid; i < 4 * kSpBins; i += kSpSmpThreads) (&sh.hist[0][0])[i] = 0;
    if (tid < 4) {
        SpCol &col = sc.col[(size_t)t * M + 4 * q + tid];
        col.cnt = 0;
        col.epoch = 0;
    }
    if (tid == 0 && q == 0) { sc.fail[t] = 0; sc.namb[t] = 0; }
    if (tid == 0) {
        const int mid = g.s / 2, q1 = g.s / 4, q3 = (3 * g.s) / 4;
        const int tk[6] = {mid - g.delta, mid + g.delta, q1 - g.delta_q, q1 + g.delta_q, q3 - g.delta_q, q3 + g.delta_q};
#pragma unroll
        for (int i = 0; i < 6; ++i) sh.tk[i] = (uint32_t)min(max(tk[i], 0), g.s - 1);
    }
    if (tid < 24) sh.tb[tid / 6][tid % 6] = 0xFFFFFFFFu;
    if (warp < 4) {
        const uint32_t key = sp_warp_sort(f2key(xpre), lane);
        const float c50 = key2f(__shfl_sync(0xFFFFFFFFu, key, 16));
        const float c25 = key2f(__shfl_sync(0xFFFFFFFFu, key, 8)), c75 = key2f(__shfl_sync(0xFFFFFFFFu, key, 23));
        if (lane == 0) {
            const float sig = (c75 - c25) / 1.35f;
            const float inv_bw = 64.0f / sig;     // 2048 bins over +-16 sigma
            const float off = (float)(1024.0 - (double)c50 * (double)inv_bw);
            sh.inv_bw[warp] = inv_bw;
            sh.off[warp] = off;
            sh.ok[warp] = (sig > 0.0f) && (inv_bw < kFltMax) && (fabsf(off) < kFltMax);
        }
    }
    __syncthreads();
    {
        float ib[4], of[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) { ib[c] = sh.ok[c] ? sh.inv_bw[c] : 0.0f; of[c] = sh.ok[c] ? sh.off[c] : 0.0f; }
#pragma unroll
        for (int j = 0; j < kSpSmpLoads; ++j) {
            if (tid + j * kSpSmpThreads < g.s) {
                const float v[4] = {xs[j].x, xs[j].y, xs[j].z, xs[j].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    int b = __float2int_rd(__fmaf_rn(v[c], ib[c], of[c]));
                    b = min(max(b, 0), kSpSBins - 1);
                    atomicAdd(&sh.hist[c][b >> 1], (b & 1) ? 0x10000u : 1u);
                }
            }
        }
    }
    __syncthreads();
    // bins of the six sample ranks: 64 threads per metric scan its 2048 bin counts, WPT words (2 bins each) per thread
    const int c = tid / kSpSmpG, gt = tid % kSpSmpG, gw = gt >> 5;
    constexpr int WPT = kSpBins / kSpSmpG;
    uint32_t w[WPT], sum = 0;
#pragma unroll
    for (int i = 0; i < WPT; ++i) { w[i] = sh.hist[c][gt * WPT + i]; sum += (w[i] & 0xFFFFu) + (w[i] >> 16); }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
    if (lane == 31) sh.warp_tot[c][gw] = incl;
    __syncthreads();
    const uint32_t excl = (gw ? sh.warp_tot[c][0] : 0u) + incl - sum;
#pragma unroll 1
    for (int i6 = 0; i6 < 6; ++i6) {
        const uint32_t k = sh.tk[i6];
        if (k >= excl && k < excl + sum) {
            uint32_t run = excl;
#pragma unroll
            for (int i = 0; i < WPT; ++i) {
                const uint32_t c0 = w[i] & 0xFFFFu, c1 = w[i] >> 16;
                if (k >= run && k < run + c0) sh.tb[c][i6] = (uint32_t)(2 * (gt * WPT + i));
                run += c0;
                if (k >= run && k < run + c1) sh.tb[c][i6] = (uint32_t)(2 * (gt * WPT + i) + 1);
                run += c1;
            }
        }
    }
    __syncthreads();
    if (tid < 4) {
        const int cc = tid;
        SpCol &col = sc.col[(size_t)t * M + 4 * q + cc];
        bool ok = sh.ok[cc] != 0;
#pragma unroll
        for (int i = 0; i < 6; ++i) ok = ok && sh.tb[cc][i] != 0xFFFFFFFFu;
        float lo = 0.0f, hi = 0.0f, dlo = 0.0f, dhi = 0.0f;
        if (ok) {
            // value at the lower edge of bin b under the map x -> x * inv_bw + off
            const double inv = 1.0 / (double)sh.inv_bw[cc], offd = (double)sh.off[cc];
            auto edge = [&](uint32_t b) -> float {
                if (b == 0) return -kFltMax;
                if (b >= (uint32_t)kSpSBins) return kFltMax;
                const double e = ((double)b - offd) * inv;
                return (float)fmin(fmax(e, -(double)kFltMax), (double)kFltMax);
            };
            lo = fdown(edge(sh.tb[cc][0]));
            hi = fup(edge(sh.tb[cc][1] + 1));
            if (lo < -kFltMax) lo = -kFltMax;
            if (hi > kFltMax) hi = kFltMax;
            // The MAD is the half-width d at which [med - d, med + d] holds half of the column: the
            // span between the quartiles' outer (inner) neighbours holds more (less) than half with
            // high probability, and for a column roughly symmetric about its median the half-lengths
            // of those spans bracket d.  (A miss is caught by the counts.)
            const float a_lo = edge(sh.tb[cc][2]), a_hi = edge(sh.tb[cc][3] + 1), b_lo = edge(sh.tb[cc][4]), b_hi = edge(sh.tb[cc][5] + 1);
            const float d0 = 0.5f * (b_lo - a_hi), d1 = 0.5f * (b_hi - a_lo);
            dlo = d0 > 0.0f ? fdown(d0) : 0.0f;
            dhi = (d1 >= 0.0f && d1 < kFltMax) ? fup(d1) : kFltMax;
            if (dhi > kFltMax) dhi = kFltMax;
        }
        col.lo = lo; col.hi = hi; col.dlo = dlo; col.dhi = dhi;
        if (!ok) {
            atomicOr(&sc.fail[t], 1u);
            if (reasons) atomicAdd(reasons + kWhySelect, 1u);
        }
    }
}

// ---- 1. / 3. sweeps ----------------------------------------------------------------------------
struct SpSweepShared {
    float lo[kSpMaxM], hi[kSpMaxM], med[kSpMaxM], rlo[kSpMaxM], rhi[kSpMaxM], sgn[kSpMaxM];
    uint32_t cnt[kSpMaxM];   // elements below the interval, this CTA
    uint32_t n32[4];         // kept counts, two 16-bit fields per word (metric m: word m / 2)
    uint32_t fail;
};

// MODE 0: count x < lo, keep lo <= x <= hi.  MODE 1: the same for d = |x - med| against
// [dlo, dhi], plus the exceedance bits and the finite check.
// Kept elements: every batch (kSpU ranks x 4 metrics per thread) the lanes of a metric quad
// scan their four 8-bit kept counts (one packed word), the first lane reserves list space for
// all of them with two shared-memory atomics (16-bit counter pairs), and every lane stores
// its kept values at its own offset.  Stores past a list's capacity land in the slack behind
// it; the full list is detected from the counter.
template <int NQ, int MODE>
__global__ void __launch_bounds__(kSpThreads, 4) xsplit_sweep_kernel(const XrankArgs a, const MetricParams p, const SpGeom g,
                                                                     const SpScratch sc) {
    constexpr int M = 4 * NQ, LPI = kSpThreads / NQ;
    extern __shared__ __align__(16) uint32_t slist[];   // [M][cap + kSpSlack]
    __shared__ SpSweepShared sh;
    const int chunk = blockIdx.x, t = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const int R = a.R;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    uint8_t *maskrow = a.mask_base ? reinterpret_cast<uint8_t *>(a.mask_base) + (size_t)slot * R : nullptr;
    const int r0 = min(R, chunk * g.slice), r1 = min(R, r0 + g.slice);
    SpCol *cols = sc.col + (size_t)t * M;
    const int cap = g.cap;

    // other CTAs of the step may raise the flag while this one runs: one read, the same answer for all threads
    if (tid == M) sh.fail = sc.fail[t];
    if (tid < M) {
        const SpCol cc = cols[tid];
        sh.lo[tid] = MODE == 0 ? cc.lo : cc.dlo;
        sh.hi[tid] = MODE == 0 ? cc.hi : cc.dhi;
        sh.med[tid] = cc.med; sh.rlo[tid] = cc.rlo; sh.rhi[tid] = cc.rhi;
        sh.sgn[tid] = p.dir[tid] < 0 ? -1.0f : 1.0f;
        sh.cnt[tid] = 0;
    }
    if (tid < 4) sh.n32[tid] = 0u;
    // this CTA's part of the exceedance row starts at zero; bits are OR-ed in
    __syncthreads();
    if (sh.fail) return;
    if (MODE == 1 && maskrow) {
        for (int i = r0 + 4 * tid; i < r1; i += 4 * kSpThreads) *reinterpret_cast<uint32_t *>(maskrow + i) = 0u;
        __syncthreads();   // zeroed before any thread ORs a bit in
    }

    const int q = tid & (NQ - 1), rl = tid / NQ;
    float lo[4], hi[4], sg[4], nsm[4], rlo[4];
    uint32_t cnt[4] = {0, 0, 0, 0};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int m = 4 * q + c;
        lo[c] = sh.lo[m]; hi[c] = sh.hi[m];
        if (MODE == 0) {
            sg[c] = 0.0f; nsm[c] = 0.0f; rlo[c] = 0.0f;
        } else {
            sg[c] = sh.sgn[m];
            nsm[c] = -sg[c] * sh.med[m];
            rlo[c] = sh.rlo[m];
        }
    }
    const uint32_t pitch = (uint32_t)(cap + kSpSlack) * 4u;   // bytes between the lists of consecutive metrics
    const uint32_t list_s = (uint32_t)__cvta_generic_to_shared(slist) + (uint32_t)(4 * q) * pitch;
    const uint32_t n32_s = (uint32_t)__cvta_generic_to_shared(&sh.n32[2 * q]);
    const uint32_t cap16 = (uint32_t)cap | ((uint32_t)cap << 16);

    auto batch = [&](const int base, const bool guard) {
        float v[kSpU][4];
        const float4 *src = reinterpret_cast<const float4 *>(row + (size_t)(base + rl) * M) + q;
#pragma unroll
        for (int j = 0; j < kSpU; ++j) {
            float4 x = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (!guard || base + j * LPI + rl < r1) x = __ldg(src + (size_t)j * LPI * NQ);
            v[j][0] = x.x; v[j][1] = x.y; v[j][2] = x.z; v[j][3] = x.w;
        }
        if (guard) {   // ranks beyond the end: +inf is neither below nor inside any interval; never "slow"
#pragma unroll
            for (int j = 0; j < kSpU; ++j)
                if (base + j * LPI + rl >= r1) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) v[j][c] = MODE == 0 ? CUDART_INF_F : __fmul_rn(sg[c], -nsm[c]);   // MODE 1: x = med
                }
        }
        uint32_t packed = 0;
#pragma unroll
        for (int j = 0; j < kSpU; ++j) {
            if (MODE == 1) {
                // d = |x - med| (one rounding, the sign of the bad direction folded in).  One test per
                // element catches everything the common path cannot decide: d beyond the lower end of
                // the threshold's range (a possible exceedance) and values that are not finite (the
                // comparison is false for NaN).
                bool slow = false;
                float sdev[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    sdev[c] = __fmaf_rn(v[j][c], sg[c], nsm[c]);
                    const float d = fabsf(sdev[c]);
                    v[j][c] = d;
                    slow |= !(d <= rlo[c]);
                }
                // The rare remainder, settled while the signed deviations are at hand (no reload): the
                // finite check, then exact tests against the threshold's possible range [rlo, rhi]; the
                // bit is set at once or the decision deferred until the MAD is known.
                if (slow) {
                    const int r = base + j * LPI + rl;
                    if (!guard || r < r1) {
                        uint32_t eb = 0;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int m = 4 * q + c;
                            // a deviation that is not finite: the value itself (re-read, this is rare) decides,
                            // since two finite values of opposite sign may differ by more than the largest float
                            if (!(fabsf(sdev[c]) <= kFltMax) && a.check_finite &&
                                nonfinite_bits(__float_as_uint(__ldg(row + (size_t)r * M + m))))
                                atomicOr(a.status, kStatNonFinite);
                            if (sdev[c] > rlo[c]) {
                                if (sdev[c] > sh.rhi[m]) {
                                    eb |= 1u << m;
                                } else {
                                    const uint32_t pos = atomicAdd(sc.namb + t, 1u);
                                    if (pos < (uint32_t)kSpAmb) sc.amb[(size_t)t * kSpAmb + pos] = ((uint32_t)r << 5) | (uint32_t)m;
                                }
                            }
                        }
                        if (eb && maskrow) atomicOr(reinterpret_cast<unsigned int *>(maskrow + (r & ~3)), eb << (8 * (r & 3)));
                    }
                }
                if (guard && base + j * LPI + rl >= r1) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) v[j][c] = CUDART_INF_F;
                }
            }
            sp_cell_count<1u>(v[j][0], lo[0], hi[0], cnt[0], packed);
            sp_cell_count<1u << 8>(v[j][1], lo[1], hi[1], cnt[1], packed);
            sp_cell_count<1u << 16>(v[j][2], lo[2], hi[2], cnt[2], packed);
            sp_cell_count<1u << 24>(v[j][3], lo[3], hi[3], cnt[3], packed);
        }
        // inclusive scan of the four 8-bit kept counts over the lanes of the same metric quad
        uint32_t incl = packed;
#pragma unroll
        for (int d = NQ; d < 32; d <<= 1) sp_scan_step(incl, d);
        const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 32 - NQ + q);
        uint32_t b01 = 0, b23 = 0;
        if (lane < NQ) {
            b01 = sp_atoms_add(n32_s, __byte_perm(total, 0, 0x4140));
            b23 = sp_atoms_add(n32_s + 4, __byte_perm(total, 0, 0x4342));
        }
        b01 = __shfl_sync(0xFFFFFFFFu, b01, q);
        b23 = __shfl_sync(0xFFFFFFFFu, b23, q);
        const uint32_t excl = incl - packed;
        // list positions of this thread's first kept element per metric (two 16-bit fields per word), clamped
        const uint32_t p01 = __vminu2(b01 + __byte_perm(excl, 0, 0x4140), cap16);
        const uint32_t p23 = __vminu2(b23 + __byte_perm(excl, 0, 0x4342), cap16);
        uint32_t addr[4];
        addr[0] = list_s + 4u * (p01 & 0xFFFFu);
        addr[1] = list_s + pitch + 4u * (p01 >> 16);
        addr[2] = list_s + 2u * pitch + 4u * (p23 & 0xFFFFu);
        addr[3] = list_s + 3u * pitch + 4u * (p23 >> 16);
#pragma unroll
        for (int j = 0; j < kSpU; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) sp_cell_keep(v[j][c], lo[c], hi[c], addr[c]);
    };
    const int span = LPI * kSpU;
    int base = r0;
    for (; base + span <= r1; base += span) batch(base, false);
    if (base < r1) batch(base, true);
    // counts below the interval: summed over the lanes of a quad class, then over the CTA
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int tot = group_sum<NQ>((int)cnt[c]);
        if (lane < NQ && tot) atomicAdd(&sh.cnt[4 * q + c], (uint32_t)tot);
    }
    __syncthreads();
    // this CTA's counts and kept elements join the step's
    // (every CTA has its own segment of the step's lists: plain stores, nothing to wait for)
    if (tid < M) {
        const uint32_t nl = (sh.n32[tid >> 1] >> (16 * (tid & 1))) & 0xFFFFu;
        if (sh.cnt[tid]) atomicAdd(&cols[tid].cnt, sh.cnt[tid]);
        sc.nseg[((size_t)t * M + tid) * g.chunks + chunk] = nl;
        if (nl > (uint32_t)cap) atomicOr(&sc.fail[t], 1u);
    }
#pragma unroll 1
    for (int m = 0; m < M; ++m) {
        const uint32_t nl = min((sh.n32[m >> 1] >> (16 * (m & 1))) & 0xFFFFu, (uint32_t)cap);
        uint32_t *dst = sc.list + (((size_t)t * M + m) * g.chunks + chunk) * cap;
        const uint32_t *srcl = slist + (size_t)m * (cap + kSpSlack);
        for (uint32_t i = tid; i < nl; i += kSpThreads) dst[i] = srcl[i];
    }
}

// ---- 2. / 4. selections ------------------------------------------------------------------------
// Finds the bin of hist[kSpBins] holding 0-based rank k (all threads of the CTA).
__device__ __forceinline__ void sp_find_bin(SpSelShared &sh, uint32_t k) {
    constexpr int G = kSpSelThreads, BPT = kSpBins / G;
    const int tid = threadIdx.x, lane = tid & 31, gw = tid >> 5;
    uint32_t loc[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) { loc[i] = sh.hist[tid * BPT + i]; sum += loc[i]; }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
    if (lane == 31) sh.warp_tot[gw] = incl;
    if (tid == 0) sh.found = 0;
    __syncthreads();
    uint32_t off = 0;
    for (int w = 0; w < gw; ++w) off += sh.warp_tot[w];
    const uint32_t excl = off + incl - sum;
    if (k >= excl && k < excl + sum) {
        uint32_t run = excl;
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            if (k >= run && k < run + loc[i]) { sh.bin = (uint32_t)(tid * BPT + i); sh.before = run; sh.cnt = loc[i]; sh.found = 1; }
            run += loc[i];
        }
    }
    __syncthreads();
}

// Keys of ranks k and (if want_next) k + 1 among the n kept elements of a column (raw float
// bits in global scratch, one segment per sweep CTA), all of whose keys lie in [base, base +
// width].  The elements are fetched once into registers (JMAX per thread).  A 1024-bin histogram over the interval
// locates the bin of rank k; while that bin holds more than 32 keys it becomes the next,
// narrower range; then the bin's keys are gathered and one warp ranks them.  The next order
// statistic is the following gathered key or, if the bin ends there, the smallest key above it.
template <int JMAX>
__device__ bool sp_select_regs(const uint32_t *__restrict__ list, const int cap, const uint32_t (&nseg)[kSpSegs], uint32_t k,
                               bool want_next, uint32_t base, uint32_t width, SpSelShared &sh, uint32_t &v1, uint32_t &v2) {
    constexpr int G = kSpSelThreads, JS = JMAX / kSpSegs;   // registers per segment
    const int tid = threadIdx.x;
    uint32_t off[JMAX];   // key - base; 0xFFFFFFFF (beyond any width) where there is no element
#pragma unroll
    for (int sg = 0; sg < kSpSegs; ++sg)
#pragma unroll
        for (int j = 0; j < JS; ++j) {
            const uint32_t i = (uint32_t)(tid + j * G);
            off[sg * JS + j] = 0x7F800000u;   // bits of +inf: its key lies above every finite key
            if (i < nseg[sg]) off[sg * JS + j] = list[(size_t)sg * cap + i];
        }
#pragma unroll
    for (int j = 0; j < JMAX; ++j) {
        const uint32_t key = key_of_bits(off[j]);
        off[j] = key >= base ? key - base : 0xFFFFFFFFu;
    }
    uint32_t krem = k;
    bool ok = true;
    v1 = v2 = 0;
    for (int round = 0; round < 4; ++round) {
        const int bits = 32 - __clz(width);
        const int shv = bits > 10 ? bits - 10 : 0;
        for (int i = tid; i < kSpBins; i += G) sh.hist[i] = 0;
        if (tid == 0) { sh.scount = 0; sh.vmin = 0xFFFFFFFFu; }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < JMAX; ++j)
            if (off[j] <= width) atomicAdd(&sh.hist[off[j] >> shv], 1u);
        __syncthreads();
        sp_find_bin(sh, krem);
        if (!sh.found) { ok = false; break; }
        krem -= sh.before;
        const uint32_t bin = sh.bin, cnt = sh.cnt;
        if (cnt <= 32u || shv == 0) {
            if (shv == 0) {   // the bin is a single key
                v1 = base + bin;
                v2 = v1;
                if (!(want_next && krem + 1 >= cnt)) break;
            }
            // gather the bin's keys, and the smallest key above the bin
            uint32_t mn = 0xFFFFFFFFu;
#pragma unroll
            for (int j = 0; j < JMAX; ++j) {
                if (off[j] <= width) {
                    const uint32_t b = off[j] >> shv;
                    if (b == bin && shv != 0) {
                        const uint32_t pos = atomicAdd(&sh.scount, 1u);
                        if (pos < 32u) sh.small[pos] = off[j];
                    } else if (b > bin) {
                        mn = min(mn, off[j]);
                    }
                }
            }
            mn = __reduce_min_sync(0xFFFFFFFFu, mn);
            if ((tid & 31) == 0 && mn != 0xFFFFFFFFu) atomicMin(&sh.vmin, mn);
            __syncthreads();
            if (shv == 0) {
                v2 = sh.vmin == 0xFFFFFFFFu ? 0xFFFFFFFFu : base + sh.vmin;
                if (sh.vmin == 0xFFFFFFFFu) ok = false;
                break;
            }
            if (tid < 32) {   // rank the gathered keys (ties by position): ranks krem and krem + 1
                const uint32_t mine = (uint32_t)tid < cnt ? sh.small[tid] : 0xFFFFFFFFu;
                uint32_t rank = 0;
                for (uint32_t j = 0; j < cnt; ++j) {
                    const uint32_t o = sh.small[j];
                    rank += (o < mine) || (o == mine && j < (uint32_t)tid);
                }
                if ((uint32_t)tid < cnt && rank == krem) sh.r1 = mine;
                if ((uint32_t)tid < cnt && rank == krem + 1) sh.r2 = mine;
            }
            __syncthreads();
            v1 = base + sh.r1;
            if (krem + 1 < cnt) v2 = base + sh.r2;
            else if (sh.vmin != 0xFFFFFFFFu) v2 = base + sh.vmin;
            else { v2 = v1; if (want_next) ok = false; }
            break;
        }
        base += bin << shv;
        // re-base the offsets on the chosen bin: keys outside it drop out
#pragma unroll
        for (int j = 0; j < JMAX; ++j) {
            const uint32_t o = off[j];
            off[j] = (o <= width && (o >> shv) == bin) ? o - (bin << shv) : 0xFFFFFFFFu;
        }
        width = (1u << shv) - 1u;
        __syncthreads();
        if (round == 3) ok = false;
    }
    __syncthreads();
    return ok;
}

template <int MODE>
__global__ void __launch_bounds__(kSpSelThreads, 12) xsplit_select_kernel(const XrankArgs a, const MetricParams p, const SpGeom g,
                                                                      const SpScratch sc, uint32_t *reasons) {
    __shared__ SpSelShared sh;
    __shared__ uint32_t s_fail;
    const int m = blockIdx.x, t = blockIdx.y, tid = threadIdx.x;
    if (tid == 0) s_fail = sc.fail[t];   // other columns of the step may raise it meanwhile: one read for all threads
    __syncthreads();
    if (s_fail) return;
    const int R = a.R, M = a.M;
    const size_t so = (size_t)t * M;
    SpCol &col = sc.col[so + m];
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2), k2 = (uint32_t)(R / 2);
    const uint32_t clt = col.cnt;
    uint32_t nseg[kSpSegs], n = 0;
    bool over = false;
#pragma unroll
    for (int sg = 0; sg < kSpSegs; ++sg) {
        nseg[sg] = sg < g.chunks ? sc.nseg[(so + m) * g.chunks + sg] : 0u;
        over |= nseg[sg] > (uint32_t)g.cap;
        n += nseg[sg];
    }
    const float flo = MODE == 0 ? col.lo : col.dlo, fhi = MODE == 0 ? col.hi : col.dhi;
    int why = -1;
    if (over) why = kWhyCtaList;
    else if (clt > k1 || k2 >= clt + n) why = MODE == 0 ? kWhyMedianMiss : kWhyMadMiss;
    if (MODE == 1 && sc.namb[t] > (uint32_t)kSpAmb) why = kWhyAmbList;
    uint32_t v1 = 0, v2 = 0;
    if (why < 0) {
        const uint32_t base = f2key((MODE == 0 && flo == 0.0f) ? -0.0f : flo);
        const uint32_t width = f2key((MODE == 0 && fhi == 0.0f) ? 0.0f : fhi) - base;
        // short lists (the brackets from the previous block's records keep about half as much as sampled ones)
        // take the selection with fewer registers per thread: the same steps over fewer slots
        bool small = true;
#pragma unroll
        for (int sg = 0; sg < kSpSegs; ++sg) small = small && nseg[sg] <= (uint32_t)((kSpJsmall / kSpSegs) * kSpSelThreads);
        const uint32_t *lst = sc.list + (so + m) * g.chunks * g.cap;
        const bool sel = small ? sp_select_regs<kSpJsmall>(lst, g.cap, nseg, k1 - clt, even, base, width, sh, v1, v2)
                               : sp_select_regs<kSpJmax>(lst, g.cap, nseg, k1 - clt, even, base, width, sh, v1, v2);
        if (!sel) why = kWhySelect;
    }
    if (tid == 0) {
        if (why < 0) {
            const float val = median_from_keys(v1, v2, even);
            if (MODE == 0) {
                a.med[so + m] = val;
                if (a.med_user) a.med_user[so + m] = val;
                const float rel = __fmul_rn(p.floor_rel[m], fabsf(val));
                col.med = val;
                col.rlo = __fmul_rn(p.thrp[m], fmaxf(fmaxf(col.dlo, rel), p.floor_abs[m]));
                col.rhi = __fmul_rn(p.thrp[m], fmaxf(fmaxf(col.dhi, rel), p.floor_abs[m]));
                col.cnt = 0;   // the MAD sweep counts anew
            } else {
                a.mad[so + m] = val;
                if (a.mad_user) a.mad_user[so + m] = val;
                col.rhs = __fmul_rn(p.thrp[m], scale_of(val, col.med, p.floor_rel[m], p.floor_abs[m]));
                col.mad = val;
                col.epoch = sc.epoch;
            }
        } else {
            atomicOr(&sc.fail[t], 1u);
            if (reasons) atomicAdd(reasons + why, 1u);
        }
    }
}

// ---- 5. finish ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSpThreads) xsplit_finish_kernel(const XrankArgs a, const MetricParams p, const SpScratch sc) {
    extern __shared__ uint32_t fhist[];   // M * 256 words for the direct path
    __shared__ XrShared xsh;
    const int t = blockIdx.x, tid = threadIdx.x;
    const int R = a.R, M = a.M;
    if (sc.fail[t]) {   // the direct radix select recomputes the whole step
        xrank_direct_step(a, p, t, fhist, xsh);
        if (tid == 0 && a.fallbacks) atomicAdd(a.fallbacks, 1u);
        return;
    }
    if (!a.mask_base) return;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    uint8_t *maskrow = reinterpret_cast<uint8_t *>(a.mask_base) + (size_t)slot * R;
    const SpCol *cols = sc.col + (size_t)t * M;
    const uint32_t na = sc.namb[t];
    for (uint32_t i = tid; i < na; i += kSpThreads) {
        const uint32_t e = sc.amb[(size_t)t * kSpAmb + i];
        const uint32_t r = e >> 5, m = e & 31u;
        if (exceeds(row[(size_t)r * M + m], cols[m].med, p.dir[m], cols[m].rhs)) {
            unsigned int *w = reinterpret_cast<unsigned int *>(maskrow + (r & ~3u));
            atomicOr(w, (1u << m) << (8 * (r & 3u)));
        }
    }
}

// Kept fraction of a column: the median interval spans 2 delta of s sample ranks, the MAD
// interval 4 delta_q (one band around each quartile), plus the bins the interval ends are
// rounded to.
SpGeom split_geometry(int R) {
    SpGeom g{};
    g.chunks = (R + kSpSlice - 1) / kSpSlice;
    g.slice = ((R + g.chunks - 1) / g.chunks + 15) / 16 * 16;
    g.stride = (R + kSpSample - 1) / kSpSample;
    if (g.stride < 1) g.stride = 1;
    g.s = 4 * (R / (4 * g.stride));
    const double sq = sqrt((double)g.s);
    // half-widths in sample ranks: 5.5 standard deviations of the sampled median's rank; the quartile
    // intervals bracket a count, the sum of two quartile ranks (sd ~ 0.61 sqrt(s)), at 5 standard deviations
    g.delta = (int)ceil(5.5 * 0.5 * sq);
    g.delta_q = (int)ceil(0.5 * 5.0 * 0.612 * sq);
    const double f_med = 2.0 * g.delta / g.s, f_mad = 4.0 * g.delta_q / g.s;
    const double f = (f_med > f_mad ? f_med : f_mad) + 0.02;
    g.cap = (int)ceil(g.slice * f * 1.2) + 64;
    g.cap = (g.cap + 31) / 32 * 32;
    if (g.cap < 256) g.cap = 256;
    return g;
}

size_t split_sweep_smem(const SpGeom &g, int M) { return (size_t)M * (g.cap + kSpSlack) * sizeof(uint32_t); }

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

bool xrank_split_supported(int R, int M) {
    if (M != 4 && M != 8) return false;
    if (R < 4096 || (R & 3) != 0) return false;
    const SpGeom g = split_geometry(R);
    if (g.slice > 32768) return false;
    // the register selection holds a whole column's kept elements: kSpJmax / kSpSegs per thread and segment
    if (g.chunks > kSpSegs || g.cap > (kSpJmax / kSpSegs) * kSpSelThreads) return false;
    return split_sweep_smem(g, M) <= 64 * 1024;
}

size_t xrank_split_scratch_bytes(int R, int M, int S_max) {
    const SpGeom g = split_geometry(R);
    size_t b = 0;
    b += align256((size_t)S_max * M * sizeof(SpCol));
    b += align256((size_t)S_max * sizeof(uint32_t)) * 2;
    b += align256((size_t)S_max * kSpAmb * sizeof(uint32_t));
    b += align256((size_t)S_max * M * g.chunks * sizeof(uint32_t));
    b += align256((size_t)S_max * M * g.chunks * g.cap * sizeof(uint32_t));
    return b;
}

cudaError_t launch_xrank_split(const XrankArgs &a, const MetricParams &p, int S, void *scratch, uint32_t *reasons,
                               cudaStream_t st, std::vector<std::pair<cudaEvent_t, cudaEvent_t>> *prof) {
    if (S <= 0) return cudaSuccess;
    const int M = a.M;
    const SpGeom g = split_geometry(a.R);
    SpScratch sc{};
    char *b = (char *)scratch;
    sc.col = (SpCol *)b;      b += align256((size_t)S * M * sizeof(SpCol));
    sc.fail = (uint32_t *)b;  b += align256((size_t)S * sizeof(uint32_t));
    sc.namb = (uint32_t *)b;  b += align256((size_t)S * sizeof(uint32_t));
    sc.amb = (uint32_t *)b;   b += align256((size_t)S * kSpAmb * sizeof(uint32_t));
    sc.nseg = (uint32_t *)b;  b += align256((size_t)S * M * g.chunks * sizeof(uint32_t));
    sc.list = (uint32_t *)b;
    sc.epoch = a.hint_epoch;
    const size_t smem = split_sweep_smem(g, M);
    static std::mutex attr_mutex;
    static bool attr_set_dev[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(attr_mutex);
    bool &attr_set = attr_set_dev[dev & 63];
    if (!attr_set) {
        e = cudaFuncSetAttribute(xsplit_sweep_kernel<2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(xsplit_sweep_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(xsplit_sweep_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(xsplit_sweep_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (prof && (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess)) return cudaGetLastError();
    const dim3 gcol(M, S), gsw(g.chunks, S);
    xsplit_sample_kernel<<<dim3(M / 4, S), kSpSmpThreads, 0, st>>>(a, g, sc, reasons);
    if (M == 8) xsplit_sweep_kernel<2, 0><<<gsw, kSpThreads, smem, st>>>(a, p, g, sc);
    else xsplit_sweep_kernel<1, 0><<<gsw, kSpThreads, smem, st>>>(a, p, g, sc);
    xsplit_select_kernel<0><<<gcol, kSpSelThreads, 0, st>>>(a, p, g, sc, reasons);
    if (prof) cudaEventRecord(ev0, st);   // the MAD / exceedance sweep, the longest kernel of the six
    if (M == 8) xsplit_sweep_kernel<2, 1><<<gsw, kSpThreads, smem, st>>>(a, p, g, sc);
    else xsplit_sweep_kernel<1, 1><<<gsw, kSpThreads, smem, st>>>(a, p, g, sc);
    if (prof) cudaEventRecord(ev1, st);
    xsplit_select_kernel<1><<<gcol, kSpSelThreads, 0, st>>>(a, p, g, sc, reasons);
    xsplit_finish_kernel<<<S, kSpThreads, (size_t)M * 256 * sizeof(uint32_t), st>>>(a, p, sc);
    e = cudaGetLastError();
    if (prof) prof->emplace_back(ev0, ev1);
    return e;
}

}  // namespace guard
