// Cross-rank selection, bracketed path (large fleets, metric count 4, 8, 16 or 32).
//
// A radix select sweeps every column eight times (four digits each for the median and
// the MAD).  For a large fleet almost all of that work is spent on elements that are
// nowhere near the middle.  This path brackets the wanted order statistic first and then
// touches every element once per statistic:
//
//   1. sample kernel   one CTA per step; each warp sorts a strided sample of one column in
//                      registers (bitonic network over shuffles) and derives [lo, hi], a value
//                      interval that holds the column's two middle elements with high
//                      probability, and [dlo, dhi], the same for the MAD;
//   2. median sweep    many CTAs per step stream the row with 128-bit loads: every element is
//                      counted if below lo and collected if inside [lo, hi];
//   3. median select   one CTA per column checks the counts (they prove whether the interval
//                      really holds the middle elements) and selects the exact median among the
//                      collected elements: histogram of order-preserving keys over the
//                      interval, refined until a bin is a single key;
//   4. MAD sweep       the same for |x - med| against [dlo, dhi]; in the same sweep every
//                      element's exceedance bit is decided when it is clear of the possible
//                      range of the threshold and deferred to a short list when it is not;
//   5. MAD select      exact MAD, then the threshold is fixed and the deferred elements settled;
//   6. any step whose interval failed (counts disagree, a list overflowed) is flagged and
//                      recomputed by the direct radix-select kernel, so results are always
//                      exact; the intervals only decide how fast they arrive.
//
// No CTA ever waits for another: cross-CTA combination uses atomic counters, and the kernel
// boundary orders the phases.
#include "kernels.h"
#include "xrank_common.cuh"

namespace guard {

namespace {

constexpr int kBrThreads = 256;
constexpr int kRPT = 8;              // ranks per thread in the streaming kernels
constexpr int kCtaCandTotal = 5120;  // candidate slots staged in shared memory per CTA, shared out over the metrics
constexpr int kCtaAmb = 512;         // deferred exceedance decisions staged per CTA
constexpr int kSelThreads = 256;
constexpr int kSelBins = 2048;

// ---------------------------------------------------------------------------------------
// 1. sample kernel: one warp per metric sorts 32 * EPL sampled keys in registers
// ---------------------------------------------------------------------------------------
template <int EPL>
__global__ void __launch_bounds__(1024) xrank_sample_kernel(const XrankArgs a, const XrankScratch sc, const int delta) {
    constexpr int s = 32 * EPL;
    extern __shared__ uint32_t keys[];  // [M][s], sorted per metric
    const int t = blockIdx.x, lane = lane_id(), m = warp_id();
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const int stride = R / s;
    uint32_t v[EPL];
#pragma unroll
    for (int j = 0; j < EPL; ++j) {
        const int r = (lane * EPL + j) * stride + (stride >> 1);
        v[j] = f2key(__ldg(row + (size_t)r * M + m));
    }
    warp_bitonic_sort<EPL>(v, lane);
    uint32_t *k = keys + m * s;
#pragma unroll
    for (int j = 0; j < EPL; ++j) k[lane * EPL + j] = v[j];
    __syncwarp();
    const int mid = s >> 1;
    const int ilo = max(0, mid - delta), ihi = min(s - 1, mid + delta);
    const float lo = key2f(k[ilo]), hi = key2f(k[ihi]);
    const float c = key2f(k[mid]);
    // interval of the MAD from the sample's deviations about its own median:
    // f(d) = #{x : |x - c| <= d}; dlo = largest sampled deviation with f <= ilo,
    // dhi = smallest with f >= ihi + 1.
    float dlo = 0.0f, dhi = CUDART_INF_F;
    for (int i = lane; i < s; i += 32) {
        const float d = fabsf(key2f(k[i]) - c);
        const uint32_t ka = f2key(c - d), kb = f2key(c + d);
        int lb = 0, n = s;      // lb = #{key < ka}
        while (n > 0) { const int h = n >> 1; if (k[lb + h] < ka) { lb += h + 1; n -= h + 1; } else n = h; }
        int ub = 0; n = s;      // ub = #{key <= kb}
        while (n > 0) { const int h = n >> 1; if (k[ub + h] <= kb) { ub += h + 1; n -= h + 1; } else n = h; }
        const int f = ub - lb;
        if (f <= ilo) dlo = fmaxf(dlo, d);
        if (f >= ihi + 1) dhi = fminf(dhi, d);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        dlo = fmaxf(dlo, __shfl_xor_sync(0xFFFFFFFFu, dlo, o));
        dhi = fminf(dhi, __shfl_xor_sync(0xFFFFFFFFu, dhi, o));
    }
    if (lane == 0) {
        const size_t o = (size_t)t * M + m;
        sc.lo[o] = lo;
        sc.hi[o] = hi;
        // The MAD interval was measured about the sample's median.  Moving the centre to the
        // exact median changes the count inside +-d only to second order (what one side gains
        // the other loses), so the interval is kept, opened by one ulp.
        sc.dlo[o] = dlo > 0.0f ? fdown(dlo) : 0.0f;
        sc.dhi[o] = dhi < CUDART_INF_F ? fup(dhi) : dhi;
    }
}

// ---------------------------------------------------------------------------------------
// 2./4. streaming kernels
// ---------------------------------------------------------------------------------------
// MODE 0: median sweep.  MODE 1: MAD + exceedance sweep.
template <int NQ, int MODE, typename MaskT>
__global__ void __launch_bounds__(kBrThreads) xrank_stream_kernel(const XrankArgs a, const MetricParams p,
                                                                 const XrankScratch sc) {
    constexpr int M = 4 * NQ;
    constexpr int LPI = kBrThreads / NQ;       // rank lanes per iteration
    constexpr int CHUNK = LPI * kRPT;          // ranks per CTA
    constexpr int kCtaCand = kCtaCandTotal / M;
    __shared__ uint32_t s_cand[M][kCtaCand];
    __shared__ uint32_t s_cnt[M], s_ncand[M], s_base[M];
    __shared__ uint32_t s_amb[MODE == 1 ? kCtaAmb : 1];
    __shared__ uint32_t s_namb, s_ambbase;
    __shared__ int s_overflow;

    const int t = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, lane = lane_id();
    if (__ldcg(sc.flag + t) != 0) return;   // the step already goes to the direct path
    const int R = a.R;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const int q = tid & (NQ - 1), rl = tid / NQ;
    const size_t so = (size_t)t * M;

    if (tid < M) { s_cnt[tid] = 0; s_ncand[tid] = 0; }
    if (tid == 0) { s_namb = 0; s_overflow = 0; }
    __syncthreads();

    float lo[4], hi[4], med[4], rlo[4], rhi[4];
    int dirv[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int m = 4 * q + c;
        if (MODE == 0) {
            lo[c] = sc.lo[so + m];
            hi[c] = sc.hi[so + m];
        } else {
            lo[c] = sc.dlo[so + m];
            hi[c] = sc.dhi[so + m];
            med[c] = a.med[so + m];
            rlo[c] = sc.rhs_lo[so + m];
            rhi[c] = sc.rhs_hi[so + m];
            dirv[c] = p.dir[m];
        }
    }
    int cnt[4] = {0, 0, 0, 0};
    uint32_t cmask[4] = {0, 0, 0, 0};
    float v[kRPT][4];
    bool bad = false;
    const int r0 = chunk * CHUNK + rl;
#pragma unroll
    for (int j = 0; j < kRPT; ++j) {
        const int r = r0 + j * LPI;
        float4 x = make_float4(CUDART_INF_F, CUDART_INF_F, CUDART_INF_F, CUDART_INF_F);
        if (r < R) x = __ldg(reinterpret_cast<const float4 *>(row + (size_t)r * M) + q);
        v[j][0] = x.x; v[j][1] = x.y; v[j][2] = x.z; v[j][3] = x.w;
    }
#pragma unroll
    for (int j = 0; j < kRPT; ++j) {
        const int r = r0 + j * LPI;
        const bool in = r < R;
        uint32_t ebits = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float x = v[j][c];
            if (MODE == 0) {
                if (a.check_finite && in) bad |= nonfinite_bits(__float_as_uint(x));
                cnt[c] += (x < lo[c]);
                if (x >= lo[c] && x <= hi[c]) cmask[c] |= 1u << j;
            } else {
                const float dev = __fsub_rn(x, med[c]);
                const float d = in ? fabsf(dev) : CUDART_INF_F;
                v[j][c] = d;
                cnt[c] += (d < lo[c]);
                if (d >= lo[c] && d <= hi[c]) cmask[c] |= 1u << j;
                const float sdev = dirv[c] < 0 ? -dev : dev;
                if (in && sdev > rlo[c]) {
                    if (sdev > rhi[c]) {
                        ebits |= 1u << (4 * q + c);
                    } else {   // decided once the exact MAD is known
                        const uint32_t pos = atomicAdd(&s_namb, 1u);
                        if (pos < kCtaAmb) s_amb[pos] = ((uint32_t)r << 5) | (uint32_t)(4 * q + c);
                        else s_overflow = 1;
                    }
                }
            }
        }
        if (MODE == 1 && a.mask_base) {
#pragma unroll
            for (int d = 1; d < NQ; d <<= 1) ebits |= __shfl_xor_sync(0xFFFFFFFFu, ebits, d);
            if (q == 0 && in) reinterpret_cast<MaskT *>(a.mask_base)[(size_t)slot * R + r] = (MaskT)ebits;
        }
    }
    if (MODE == 0 && a.check_finite) {
        if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(a.status, kStatNonFinite);
    }
    // counts and candidates -> shared lists
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int m = 4 * q + c;
        const int tot_cnt = group_sum<NQ>(cnt[c]);
        const int n = __popc(cmask[c]);
        int excl, total;
        group_scan<NQ>(n, excl, total);
        uint32_t base = 0;
        if (lane == q) {   // first lane of the group
            if (tot_cnt) atomicAdd(&s_cnt[m], (uint32_t)tot_cnt);
            if (total) base = atomicAdd(&s_ncand[m], (uint32_t)total);
        }
        base = __shfl_sync(0xFFFFFFFFu, base, q);
        uint32_t pos = base + excl;
#pragma unroll
        for (int j = 0; j < kRPT; ++j) {
            if ((cmask[c] >> j) & 1u) {
                if (pos < kCtaCand) s_cand[m][pos] = __float_as_uint(v[j][c]);
                ++pos;
            }
        }
    }
    __syncthreads();
    // shared lists -> the step's global lists
    if (tid < M) {
        const uint32_t n = s_ncand[tid];
        if (n > kCtaCand) { s_overflow = 1; if (sc.reasons) atomicAdd(sc.reasons + kWhyCtaList, 1u); }
        if (s_cnt[tid]) atomicAdd(sc.cnt_lt + so + tid, s_cnt[tid]);
        uint32_t base = 0;
        if (n) base = atomicAdd(sc.ncand + so + tid, n);
        s_base[tid] = base;
        if (base + n > (uint32_t)sc.cap) { s_overflow = 1; if (sc.reasons) atomicAdd(sc.reasons + kWhyStepList, 1u); }
    }
    if (MODE == 1 && tid == 32) {
        const uint32_t n = min(s_namb, (uint32_t)kCtaAmb);
        uint32_t base = 0;
        if (n) base = atomicAdd(sc.namb + t, n);
        s_ambbase = base;
        if (base + n > (uint32_t)sc.amb_cap || s_namb > (uint32_t)kCtaAmb) { s_overflow = 1; if (sc.reasons) atomicAdd(sc.reasons + kWhyAmbList, 1u); }
    }
    __syncthreads();
    if (!s_overflow) {
        for (int m = 0; m < M; ++m) {
            const uint32_t n = s_ncand[m], base = s_base[m];
            uint32_t *dst = sc.cand + (so + m) * (size_t)sc.cap + base;
            for (uint32_t i = tid; i < n; i += kBrThreads) dst[i] = s_cand[m][i];
        }
        if (MODE == 1) {
            const uint32_t n = min(s_namb, (uint32_t)kCtaAmb);
            uint32_t *dst = sc.amb + (size_t)t * sc.amb_cap + s_ambbase;
            for (uint32_t i = tid; i < n; i += kBrThreads) dst[i] = s_amb[i];
        }
    } else if (tid == 0) {
        atomicExch(sc.flag + t, 1u);
    }
}

// ---------------------------------------------------------------------------------------
// 3./5. selection kernels: one CTA per (step, metric) column finishes the statistic
// ---------------------------------------------------------------------------------------
struct SelShared {
    uint32_t hist[kSelBins];
    uint32_t warp_tot[kSelThreads / 32];
    uint32_t bin, before, cnt, vmin;
    int found;
};

// Finds the bin of sh.hist that holds 0-based rank k (all threads; results in sh).
__device__ __forceinline__ void cta_find_bin(SelShared &sh, uint32_t k) {
    constexpr int BPT = kSelBins / kSelThreads;
    const int tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    uint32_t loc[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) { loc[i] = sh.hist[tid * BPT + i]; sum += loc[i]; }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
    if (lane == 31) sh.warp_tot[warp] = incl;
    if (tid == 0) sh.found = 0;
    __syncthreads();
    uint32_t off = 0;
    for (int w = 0; w < warp; ++w) off += sh.warp_tot[w];
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

// MODE 0: median of the column from the elements collected inside [lo, hi].
// MODE 1: MAD from those inside [dlo, dhi], then the deferred exceedance decisions.
template <int MODE, typename MaskT>
__global__ void __launch_bounds__(kSelThreads) xrank_select_kernel(const XrankArgs a, const MetricParams p, const XrankScratch sc) {
    __shared__ SelShared sh;
    const int m = blockIdx.x, t = blockIdx.y, tid = threadIdx.x, lane = lane_id();
    const int R = a.R, M = a.M;
    const size_t so = (size_t)t * M, col = so + m;
    const uint32_t clt = __ldcg(sc.cnt_lt + col), n = __ldcg(sc.ncand + col);
    __syncthreads();
    // leave the counters clean for the next sweep / launch (every thread has read them)
    if (tid == 0) {
        sc.cnt_lt[col] = 0;
        sc.ncand[col] = 0;
        if (MODE == 0 && m == 0) sc.namb[t] = 0;
    }
    if (__ldcg(sc.flag + t) != 0) return;
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2), k2 = (uint32_t)(R / 2);
    int why = -1;
    if (!(clt <= k1 && k2 < clt + n && n <= (uint32_t)sc.cap)) why = (MODE == 0 ? kWhyMedianMiss : kWhyMadMiss);
    uint32_t v1 = 0, v2 = 0;
    if (why < 0) {
        const uint32_t *list = sc.cand + col * (size_t)sc.cap;
        const float flo = (MODE == 0 ? sc.lo : sc.dlo)[col], fhi = (MODE == 0 ? sc.hi : sc.dhi)[col];
        // key range of the collected elements (a float compare accepts both zeros)
        uint32_t base = f2key(flo == 0.0f ? -0.0f : flo);
        uint32_t width = f2key(fhi == 0.0f ? 0.0f : fhi) - base;
        uint32_t krem = k1 - clt, ceq = 0;
        for (;;) {
            const int bits = 32 - __clz(width);
            const int shv = bits > 11 ? bits - 11 : 0;
            for (int i = tid; i < kSelBins; i += kSelThreads) sh.hist[i] = 0;
            __syncthreads();
            for (uint32_t i = tid; i < n; i += kSelThreads) {
                const uint32_t off = key_of_bits(__ldcg(list + i)) - base;
                if (off <= width) atomicAdd(&sh.hist[off >> shv], 1u);
            }
            __syncthreads();
            cta_find_bin(sh, krem);
            if (!sh.found) { why = kWhySelect; break; }
            krem -= sh.before;
            if (shv == 0) { v1 = base + sh.bin; ceq = sh.cnt; break; }
            base += sh.bin << shv;
            width = (1u << shv) - 1u;
            __syncthreads();
        }
        v2 = v1;
        if (why < 0 && even && krem + 1 >= ceq) {   // next order statistic: smallest key above v1
            if (tid == 0) sh.vmin = 0xFFFFFFFFu;
            __syncthreads();
            uint32_t cand = 0xFFFFFFFFu;
            for (uint32_t i = tid; i < n; i += kSelThreads) {
                const uint32_t key = key_of_bits(__ldcg(list + i));
                if (key > v1) cand = min(cand, key);
            }
            cand = __reduce_min_sync(0xFFFFFFFFu, cand);
            if (lane == 0 && cand != 0xFFFFFFFFu) atomicMin(&sh.vmin, cand);
            __syncthreads();
            v2 = sh.vmin;
            if (v2 == 0xFFFFFFFFu) why = kWhySelect;
        }
    }
    if (why >= 0) {
        if (tid == 0) {
            if (sc.reasons) atomicAdd(sc.reasons + why, 1u);
            atomicExch(sc.flag + t, 1u);
        }
        return;
    }
    const float val = median_from_keys(v1, v2, even);
    if (MODE == 0) {
        if (tid == 0) {
            a.med[col] = val;
            if (a.med_user) a.med_user[col] = val;
            // range of the exceedance threshold over the MAD interval
            const float rel = __fmul_rn(p.floor_rel[m], fabsf(val));
            sc.rhs_lo[col] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(sc.dlo[col], rel), p.floor_abs[m]));
            sc.rhs_hi[col] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(sc.dhi[col], rel), p.floor_abs[m]));
        }
    } else {
        const float med = a.med[col];
        if (tid == 0) {
            a.mad[col] = val;
            if (a.mad_user) a.mad_user[col] = val;
        }
        if (a.mask_base) {
            // settle the elements whose exceedance depended on the exact MAD
            const float rhs = __fmul_rn(p.thrp[m], scale_of(val, med, p.floor_rel[m], p.floor_abs[m]));
            const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
            const float *row = a.base + (size_t)slot * a.row_stride;
            const uint32_t na = __ldcg(sc.namb + t);
            for (uint32_t i = tid; i < na; i += kSelThreads) {
                const uint32_t e = __ldcg(sc.amb + (size_t)t * sc.amb_cap + i);
                if ((int)(e & 31u) != m) continue;
                const uint32_t r = e >> 5;
                if (exceeds(row[(size_t)r * M + m], med, p.dir[m], rhs)) {
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
    }
}

template <int NQ>
cudaError_t launch_phases(const XrankArgs &a, const MetricParams &p, const XrankScratch &sc, int S, cudaStream_t st) {
    constexpr int CHUNK = (kBrThreads / NQ) * kRPT;
    const int chunks = (a.R + CHUNK - 1) / CHUNK;
    const dim3 sgrid(chunks, S), cgrid(a.M, S);
    const bool wide = a.mask_bytes == 4;
    if (wide) xrank_stream_kernel<NQ, 0, uint32_t><<<sgrid, kBrThreads, 0, st>>>(a, p, sc);
    else xrank_stream_kernel<NQ, 0, uint8_t><<<sgrid, kBrThreads, 0, st>>>(a, p, sc);
    if (wide) xrank_select_kernel<0, uint32_t><<<cgrid, kSelThreads, 0, st>>>(a, p, sc);
    else xrank_select_kernel<0, uint8_t><<<cgrid, kSelThreads, 0, st>>>(a, p, sc);
    if (wide) xrank_stream_kernel<NQ, 1, uint32_t><<<sgrid, kBrThreads, 0, st>>>(a, p, sc);
    else xrank_stream_kernel<NQ, 1, uint8_t><<<sgrid, kBrThreads, 0, st>>>(a, p, sc);
    if (wide) xrank_select_kernel<1, uint32_t><<<cgrid, kSelThreads, 0, st>>>(a, p, sc);
    else xrank_select_kernel<1, uint8_t><<<cgrid, kSelThreads, 0, st>>>(a, p, sc);
    return cudaGetLastError();
}

}  // namespace

bool xrank_bracket_supported(int R, int M) { return (M == 4 || M == 8 || M == 16 || M == 32) && R >= 4096; }

int xrank_cand_cap(int R) {
    int cap = R / 4;
    return cap < 1024 ? 1024 : cap;
}

int xrank_amb_cap(int R, int M) {
    long long c = (long long)R * M / 16;
    return (int)(c < 1024 ? 1024 : (c > (1 << 20) ? (1 << 20) : c));
}

int xrank_scratch_steps(int R, int M, int want) {
    const long long per_step = (long long)M * xrank_cand_cap(R) * 4 + (long long)xrank_amb_cap(R, M) * 4;
    long long s = (96LL << 20) / per_step;
    if (s > 256) s = 256;
    if (s > want) s = want;
    return (int)(s < 1 ? 1 : s);
}

size_t xrank_scratch_small_bytes(int M, int S_max) {
    return (size_t)S_max * (2 * M + 2) * sizeof(uint32_t);
}

size_t xrank_scratch_big_bytes(int R, int M, int S_max) {
    return (size_t)S_max * M * 6 * sizeof(float) + (size_t)S_max * M * xrank_cand_cap(R) * 4 +
           (size_t)S_max * xrank_amb_cap(R, M) * 4;
}

XrankScratch carve_xrank_scratch(void *small_base, void *big_base, int R, int M, int S_max) {
    XrankScratch sc{};
    sc.S_max = S_max;
    sc.cap = xrank_cand_cap(R);
    sc.amb_cap = xrank_amb_cap(R, M);
    uint32_t *u = (uint32_t *)small_base;   // zero-initialised state
    sc.cnt_lt = u; u += (size_t)S_max * M;
    sc.ncand = u;  u += (size_t)S_max * M;
    sc.flag = u;   u += S_max;
    sc.namb = u;
    float *f = (float *)big_base;
    sc.lo = f;     f += (size_t)S_max * M;
    sc.hi = f;     f += (size_t)S_max * M;
    sc.dlo = f;    f += (size_t)S_max * M;
    sc.dhi = f;    f += (size_t)S_max * M;
    sc.rhs_lo = f; f += (size_t)S_max * M;
    sc.rhs_hi = f; f += (size_t)S_max * M;
    sc.cand = (uint32_t *)f;
    sc.amb = sc.cand + (size_t)S_max * M * sc.cap;
    return sc;
}

// Runs the bracketed path on S <= scratch.S_max steps (sample, then one streaming sweep and
// one per-column selection for the median and again for the MAD), then the direct kernel on
// the steps it flagged.  a.med / a.mad must hold S * M floats.  Six launches.
cudaError_t launch_xrank_bracketed(const XrankArgs &a, const MetricParams &p, const XrankScratch &sc, int S,
                                   cudaStream_t st) {
    if (S <= 0) return cudaSuccess;
    const int epl = a.M <= 8 ? 32 : (a.M == 16 ? 16 : 8);
    const int s = 32 * epl;
    // half-width of the sampled interval in sample ranks: 5.5 standard deviations of a sample
    // quantile's rank (0.5 sqrt(s)), so that a miss (and the slow direct redo) is a ~1e-7 event
    const int delta = (int)ceil(5.5 * 0.5 * sqrt((double)s));
    const size_t smem = (size_t)s * a.M * sizeof(uint32_t);
    if (epl == 32) xrank_sample_kernel<32><<<S, 32 * a.M, smem, st>>>(a, sc, delta);
    else if (epl == 16) xrank_sample_kernel<16><<<S, 32 * a.M, smem, st>>>(a, sc, delta);
    else xrank_sample_kernel<8><<<S, 32 * a.M, smem, st>>>(a, sc, delta);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    switch (a.M) {
        case 4: e = launch_phases<1>(a, p, sc, S, st); break;
        case 8: e = launch_phases<2>(a, p, sc, S, st); break;
        case 16: e = launch_phases<4>(a, p, sc, S, st); break;
        case 32: e = launch_phases<8>(a, p, sc, S, st); break;
        default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
    XrankArgs d = a;
    d.only_flagged = sc.flag;
    return launch_xrank_direct(d, p, S, st);
}

}  // namespace guard
