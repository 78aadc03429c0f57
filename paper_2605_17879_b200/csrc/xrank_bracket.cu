// Cross-rank selection, bracketed path (large fleets, metric count 4, 8, 16 or 32).
//
// A radix select sweeps every column eight times (four digits each for the median and
// the MAD).  For a large fleet almost all of that work is spent on elements that are
// nowhere near the middle.  This path brackets the wanted order statistic first and then
// touches every element once per statistic:
//
//   1. sample kernel   one CTA per step sorts a strided sample of each column and derives
//                      [lo, hi], a value interval that contains the column's two middle
//                      elements with high probability, plus a first guess of the MAD interval;
//   2. median kernel   many CTAs per step stream the row with 128-bit loads: every element
//                      is counted if below lo and collected if inside [lo, hi]; the CTA that
//                      draws the step's last ticket checks the counts (they prove whether
//                      the interval really holds the middle elements) and selects the exact
//                      median among the few collected candidates by radix select on
//                      order-preserving keys;
//   3. MAD kernel      the same for |x - med| against [dlo, dhi]; in the same sweep every
//                      element's exceedance bit is decided when it is clear of the possible
//                      range of the threshold and deferred to a short list when it is not;
//                      the last CTA selects the exact MAD, fixes the threshold and settles the
//                      deferred elements;
//   4. any step whose interval failed (counts disagree, a list overflowed) is flagged and
//                      recomputed by the direct radix-select kernel, so results are always
//                      exact; the brackets only decide how fast they arrive.
//
// No CTA ever waits for another: cross-CTA combination uses atomic counters and a
// last-ticket finaliser.
#include <math_constants.h>

#include "kernels.h"

namespace guard {

namespace {

constexpr int kBrThreads = 256;
constexpr int kRPT = 8;           // ranks per thread in the streaming kernels
constexpr int kCtaCandTotal = 5120;  // candidate slots staged in shared memory per CTA, shared out over the metrics
constexpr int kCtaAmb = 512;      // deferred exceedance decisions staged per CTA
constexpr int kSampleThreads = 1024;

__device__ __forceinline__ float fdown(float x) { return __uint_as_float(f2key(x) == 0 ? __float_as_uint(x) : bits_of_key(f2key(x) - 1)); }
__device__ __forceinline__ float fup(float x) { return __uint_as_float(bits_of_key(f2key(x) + 1)); }

// ---------------------------------------------------------------------------------------
// 1. sample kernel
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSampleThreads) xrank_sample_kernel(const XrankArgs a, const XrankScratch sc, const int s,
                                                                      const int delta) {
    extern __shared__ uint32_t keys[];  // [M][s]
    const int t = blockIdx.x, tid = threadIdx.x;
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const int stride = R / s;
    for (int e = tid; e < s * M; e += blockDim.x) {
        const int i = e / M, m = e - i * M;
        const int r = i * stride + (stride >> 1);
        keys[m * s + i] = f2key(row[(size_t)r * M + m]);
    }
    // bitonic sort of every metric's sample (ascending)
    const int half = (s * M) >> 1;
    for (int size = 2; size <= s; size <<= 1) {
        for (int st = size >> 1; st > 0; st >>= 1) {
            __syncthreads();
            for (int e = tid; e < half; e += blockDim.x) {
                const int m = e / (s >> 1), q = e - m * (s >> 1);
                const int i = 2 * q - (q & (st - 1));
                const int j = i + st;
                uint32_t *k = keys + m * s;
                const bool asc = ((i & size) == 0);
                const uint32_t x = k[i], y = k[j];
                if ((x > y) == asc) { k[i] = y; k[j] = x; }
            }
        }
    }
    __syncthreads();
    // one warp per metric derives the intervals
    const int warp = warp_id(), lane = lane_id(), nwarps = blockDim.x >> 5;
    for (int m = warp; m < M; m += nwarps) {
        const uint32_t *k = keys + m * s;
        const int mid = s >> 1;
        const int ilo = max(0, mid - delta), ihi = min(s - 1, mid + delta);
        const float lo = key2f(k[ilo]), hi = key2f(k[ihi]);
        const float c = key2f(k[mid]);
        // interval of the MAD from the sample's deviations about its own median:
        // f(d) = #{x : |x - c| <= d}; dlo = largest sampled deviation with f <= jlo,
        // dhi = smallest with f >= jhi + 1.
        const int jlo = max(0, mid - delta), jhi = min(s - 1, mid + delta);
        float dlo = 0.0f, dhi = CUDART_INF_F;
        for (int i = lane; i < s; i += 32) {
            const float d = fabsf(key2f(k[i]) - c);
            const uint32_t ka = f2key(c - d), kb = f2key(c + d);
            int lb = 0, n = s;      // lb = #{key < ka}
            while (n > 0) { const int h = n >> 1; if (k[lb + h] < ka) { lb += h + 1; n -= h + 1; } else n = h; }
            int ub = 0; n = s;      // ub = #{key <= kb}
            while (n > 0) { const int h = n >> 1; if (k[ub + h] <= kb) { ub += h + 1; n -= h + 1; } else n = h; }
            const int f = ub - lb;
            if (f <= jlo) dlo = fmaxf(dlo, d);
            if (f >= jhi + 1) dhi = fminf(dhi, d);
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
            sc.center[o] = c;
            sc.dlo[o] = dlo;
            sc.dhi[o] = dhi;
        }
    }
}

// ---------------------------------------------------------------------------------------
// selection among the collected candidates (all threads of the CTA; list in global memory)
// ---------------------------------------------------------------------------------------
struct ListSel {
    uint32_t hist[256];
    uint32_t prefix, krem, ceq, v2, kand, kor;
    int need;
};

// Finds the keys of 0-based ranks k and (if want_next) k + 1 in list[0..n) (raw float bits).
__device__ void cta_select_list(const uint32_t *list, int n, uint32_t k, bool want_next, ListSel &ls, uint32_t &v1,
                                uint32_t &v2, bool &ok) {
    const int tid = threadIdx.x, lane = lane_id();
    if (tid == 0) { ls.kand = 0xFFFFFFFFu; ls.kor = 0u; ls.prefix = 0; ls.krem = k; ls.ceq = (uint32_t)n; ls.v2 = 0xFFFFFFFFu; ls.need = 0; }
    for (int i = tid; i < 256; i += blockDim.x) ls.hist[i] = 0;
    __syncthreads();
    uint32_t kand = 0xFFFFFFFFu, kor = 0u;
    for (int i = tid; i < n; i += blockDim.x) {
        const uint32_t key = key_of_bits(__ldcg(list + i));
        kand &= key;
        kor |= key;
    }
    kand = __reduce_and_sync(0xFFFFFFFFu, kand);
    kor = __reduce_or_sync(0xFFFFFFFFu, kor);
    if (lane == 0) { atomicAnd(&ls.kand, kand); atomicOr(&ls.kor, kor); }
    __syncthreads();
    const uint32_t diff = ls.kand ^ ls.kor;   // bits that vary among the candidates
    ok = true;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (((diff >> shift) & 255u) == 0) {   // this digit is the same for every candidate
            if (tid == 0) ls.prefix |= ls.kor & (255u << shift);
            __syncthreads();
            continue;
        }
        const uint32_t prefix = ls.prefix;
        const int nround = (n + blockDim.x - 1) / blockDim.x;
        for (int it = 0; it < nround; ++it) {
            const int i = it * blockDim.x + tid;
            bool valid = i < n;
            uint32_t key = 0;
            if (valid) {
                key = key_of_bits(__ldcg(list + i));
                if (pass > 0) valid = ((key ^ prefix) >> (shift + 8)) == 0;
            }
            const uint32_t digit = (key >> shift) & 255u;
            const unsigned peers = __match_any_sync(0xFFFFFFFFu, valid ? digit : (256u + lane));
            if (valid && lane == __ffs(peers) - 1) atomicAdd(&ls.hist[digit], __popc(peers));
        }
        __syncthreads();
        if (tid < 32) {
            // find the bin holding rank krem
            uint32_t loc[8], sum = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { loc[i] = ls.hist[lane * 8 + i]; sum += loc[i]; }
            uint32_t incl = sum;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
            const uint32_t excl = incl - sum, kk = ls.krem;
            const bool mine = (kk >= excl) && (kk < incl);
            const unsigned ball = __ballot_sync(0xFFFFFFFFu, mine);
            __syncwarp();
            for (int i = lane; i < 256; i += 32) ls.hist[i] = 0;
            if (mine) {
                uint32_t run = excl;
                int b = 7; uint32_t bef = excl, c = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { if (kk >= run && kk < run + loc[i]) { b = i; bef = run; c = loc[i]; } run += loc[i]; }
                ls.prefix |= (uint32_t)(lane * 8 + b) << shift;
                ls.krem = kk - bef;
                ls.ceq = c;
            }
            if (ball == 0 && lane == 0) ls.need = -1;   // rank not inside the list: caller flags the step
        }
        __syncthreads();
    }
    if (ls.need < 0) ok = false;
    v1 = ls.prefix;
    v2 = v1;
    if (want_next && ok) {
        // ceq counts the copies of the selected key (n if no digit varied at all)
        const bool need = (ls.krem + 1 >= ls.ceq);
        if (need) {
            uint32_t cand = 0xFFFFFFFFu;
            for (int i = tid; i < n; i += blockDim.x) {
                const uint32_t key = key_of_bits(__ldcg(list + i));
                if (key > v1) cand = min(cand, key);
            }
            cand = __reduce_min_sync(0xFFFFFFFFu, cand);
            if (lane == 0 && cand != 0xFFFFFFFFu) atomicMin(&ls.v2, cand);
            __syncthreads();
            v2 = ls.v2;
            if (v2 == 0xFFFFFFFFu) ok = false;
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------
// 2./3. streaming kernels
// ---------------------------------------------------------------------------------------
// Exclusive scan of `n` over the lanes of a warp that share the same quad index
// (lanes q, q + NQ, q + 2 NQ, ...); returns the exclusive prefix and the group total.
template <int NQ>
__device__ __forceinline__ void group_scan(int n, int &excl, int &total) {
    const int lane = lane_id();
    int incl = n;
#pragma unroll
    for (int d = NQ; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += u;
    }
    excl = incl - n;
    total = __shfl_sync(0xFFFFFFFFu, incl, 32 - NQ + (lane & (NQ - 1)));
}

template <int NQ>
__device__ __forceinline__ int group_sum(int v) {
#pragma unroll
    for (int d = NQ; d < 32; d <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// MODE 0: median sweep.  MODE 1: MAD + exceedance sweep.
template <int NQ, int MODE, typename MaskT>
__global__ void __launch_bounds__(kBrThreads) xrank_stream_kernel(const XrankArgs a, const MetricParams p,
                                                                 const XrankScratch sc, const int chunks) {
    constexpr int M = 4 * NQ;
    constexpr int LPI = kBrThreads / NQ;       // rank lanes per iteration
    constexpr int CHUNK = LPI * kRPT;          // ranks per CTA
    constexpr int kCtaCand = kCtaCandTotal / M;
    __shared__ uint32_t s_cand[M][kCtaCand];
    __shared__ uint32_t s_cnt[M], s_ncand[M], s_base[M];
    __shared__ uint32_t s_amb[MODE == 1 ? kCtaAmb : 1];
    __shared__ uint32_t s_namb, s_ambbase;
    __shared__ int s_overflow, s_last;
    __shared__ float s_val[M], s_rhs[M];
    __shared__ ListSel ls;

    const int t = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, lane = lane_id();
    const bool skip = __ldcg(sc.flag + t) != 0;   // the step already goes to the direct path
    const int R = a.R;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const int q = tid & (NQ - 1), rl = tid / NQ;
    const size_t so = (size_t)t * M;

    if (tid < M) { s_cnt[tid] = 0; s_ncand[tid] = 0; }
    if (tid == 0) { s_namb = 0; s_overflow = 0; }
    __syncthreads();

    if (!skip) {
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
    }  // !skip
    // last ticket of the step finalises (a skipped step still needs its counters cleaned)
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(sc.ticket + t, 1u) == (uint32_t)chunks - 1u);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    bool fail = __ldcg(sc.flag + t) != 0;
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2), k2 = (uint32_t)(R / 2);
    for (int m = 0; m < M && !fail; ++m) {
        const uint32_t clt = __ldcg(sc.cnt_lt + so + m), n = __ldcg(sc.ncand + so + m);
        if (!(clt <= k1 && k2 < clt + n && n <= (uint32_t)sc.cap)) {
            if (tid == 0 && sc.reasons) atomicAdd(sc.reasons + (MODE == 0 ? kWhyMedianMiss : kWhyMadMiss), 1u);
            fail = true;
            break;
        }
        uint32_t v1, v2;
        bool ok;
        cta_select_list(sc.cand + (so + m) * (size_t)sc.cap, (int)n, k1 - clt, even, ls, v1, v2, ok);
        if (!ok) {
            if (tid == 0 && sc.reasons) atomicAdd(sc.reasons + kWhySelect, 1u);
            fail = true;
            break;
        }
        if (tid == 0) s_val[m] = median_from_keys(v1, v2, even);
    }
    __syncthreads();
    if (!fail) {
        if (MODE == 0) {
            if (tid < M) {
                const int m = tid;
                const float med_m = s_val[m];
                a.med[so + m] = med_m;
                if (a.med_user) a.med_user[so + m] = med_m;
                // The MAD interval was measured about the sample's median.  Moving the centre
                // to the exact median changes the count inside +-d only to second order (what
                // one side gains the other loses), so the interval is kept, opened by one ulp.
                float dl = sc.dlo[so + m];
                dl = dl > 0.0f ? fdown(dl) : 0.0f;
                float dh = sc.dhi[so + m];
                if (dh < CUDART_INF_F) dh = fup(dh);
                sc.dlo[so + m] = dl;
                sc.dhi[so + m] = dh;
                const float rel = __fmul_rn(p.floor_rel[m], fabsf(med_m));
                sc.rhs_lo[so + m] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(dl, rel), p.floor_abs[m]));
                sc.rhs_hi[so + m] = __fmul_rn(p.thrp[m], fmaxf(fmaxf(dh, rel), p.floor_abs[m]));
            }
        } else {
            if (tid < M) {
                const int m = tid;
                const float mad = s_val[m];
                a.mad[so + m] = mad;
                if (a.mad_user) a.mad_user[so + m] = mad;
                s_rhs[m] = __fmul_rn(p.thrp[m], scale_of(mad, a.med[so + m], p.floor_rel[m], p.floor_abs[m]));
            }
            __syncthreads();
            if (a.mask_base) {
                const uint32_t n = __ldcg(sc.namb + t);
                for (uint32_t i = tid; i < n; i += kBrThreads) {
                    const uint32_t e = __ldcg(sc.amb + (size_t)t * sc.amb_cap + i);
                    const uint32_t r = e >> 5, m = e & 31u;
                    if (exceeds(row[(size_t)r * M + m], a.med[so + m], p.dir[m], s_rhs[m])) {
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
    } else if (tid == 0) {
        atomicExch(sc.flag + t, 1u);
    }
    // leave the counters clean for the next sweep / launch
    if (tid < M) { sc.cnt_lt[so + tid] = 0; sc.ncand[so + tid] = 0; }
    if (tid == 0) { sc.ticket[t] = 0; sc.namb[t] = 0; }
}

template <int NQ, int MODE>
cudaError_t launch_stream(const XrankArgs &a, const MetricParams &p, const XrankScratch &sc, int S, cudaStream_t st) {
    constexpr int CHUNK = (kBrThreads / NQ) * kRPT;
    const int chunks = (a.R + CHUNK - 1) / CHUNK;
    dim3 grid(chunks, S);
    if (a.mask_bytes == 4)
        xrank_stream_kernel<NQ, MODE, uint32_t><<<grid, kBrThreads, 0, st>>>(a, p, sc, chunks);
    else
        xrank_stream_kernel<NQ, MODE, uint8_t><<<grid, kBrThreads, 0, st>>>(a, p, sc, chunks);
    return cudaGetLastError();
}

template <int NQ>
cudaError_t launch_both(const XrankArgs &a, const MetricParams &p, const XrankScratch &sc, int S, cudaStream_t st) {
    cudaError_t e = launch_stream<NQ, 0>(a, p, sc, S, st);
    if (e != cudaSuccess) return e;
    return launch_stream<NQ, 1>(a, p, sc, S, st);
}

int sample_size(int R, int M) {
    int s = 1024;
    while (s > 64 && (s * M > 8192 || s * 4 > R)) s >>= 1;
    return s;
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
    return (size_t)S_max * (2 * M + 3) * sizeof(uint32_t);
}

size_t xrank_scratch_big_bytes(int R, int M, int S_max) {
    return (size_t)S_max * M * 7 * sizeof(float) + (size_t)S_max * M * xrank_cand_cap(R) * 4 +
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
    sc.ticket = u; u += S_max;
    sc.flag = u;   u += S_max;
    sc.namb = u;
    float *f = (float *)big_base;
    sc.lo = f;     f += (size_t)S_max * M;
    sc.hi = f;     f += (size_t)S_max * M;
    sc.center = f; f += (size_t)S_max * M;
    sc.dlo = f;    f += (size_t)S_max * M;
    sc.dhi = f;    f += (size_t)S_max * M;
    sc.rhs_lo = f; f += (size_t)S_max * M;
    sc.rhs_hi = f; f += (size_t)S_max * M;
    sc.cand = (uint32_t *)f;
    sc.amb = sc.cand + (size_t)S_max * M * sc.cap;
    return sc;
}

// Runs the bracketed path on S <= scratch.S_max steps, then the direct kernel on the
// steps it flagged.  a.med / a.mad must hold S * M floats.
cudaError_t launch_xrank_bracketed(const XrankArgs &a, const MetricParams &p, const XrankScratch &sc, int S,
                                   cudaStream_t st) {
    if (S <= 0) return cudaSuccess;
    const int s = sample_size(a.R, a.M);
    // half-width of the sampled interval in sample ranks: 5.5 standard deviations of a sample
    // quantile's rank (0.5 sqrt(s)), so that a miss (and the slow direct redo) is a ~1e-7 event
    const int delta = (int)ceil(5.5 * 0.5 * sqrt((double)s));
    xrank_sample_kernel<<<S, kSampleThreads, (size_t)s * a.M * sizeof(uint32_t), st>>>(a, sc, s, delta);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    switch (a.M) {
        case 4: e = launch_both<1>(a, p, sc, S, st); break;
        case 8: e = launch_both<2>(a, p, sc, S, st); break;
        case 16: e = launch_both<4>(a, p, sc, S, st); break;
        case 32: e = launch_both<8>(a, p, sc, S, st); break;
        default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
    XrankArgs d = a;
    d.only_flagged = sc.flag;
    return launch_xrank_direct(d, p, S, st);
}

}  // namespace guard
