// Per-series window-median machinery shared by the stand-alone window kernels (window.cu) and the
// tile kernel that fuses the window medians into the cross-rank median pass (xrank_tile.cu):
// the per-element count / keep step of the one-thread-per-series path, the selection among a
// thread's kept keys, and the whole-warp selection that finishes the series an interval missed.
#pragma once
#include <math_constants.h>

#include "colselect.cuh"
#include "kernels.h"

namespace guard {

constexpr int kWalkMax = 24;     // walk when the wanted rank is at most this far from the pivot

template <int VPL>
__device__ __forceinline__ void lane_sort(uint32_t (&v)[VPL]) {
#pragma unroll
    for (int p = 1; p < VPL; p <<= 1)
#pragma unroll
        for (int k = p; k >= 1; k >>= 1)
#pragma unroll
            for (int j = k % p; j + k < VPL; j += 2 * k)
#pragma unroll
                for (int i = 0; i < k; ++i)
                    if ((i + j) / (2 * p) == (i + j + k) / (2 * p)) {
                        const uint32_t x = v[i + j], y = v[i + j + k];
                        v[i + j] = min(x, y);
                        v[i + j + k] = max(x, y);
                    }
}

template <int VPL>
__device__ __forceinline__ uint32_t lane_pick(const uint32_t (&v)[VPL], int idx) {
    uint32_t r = v[0];
#pragma unroll
    for (int i = 1; i < VPL; ++i) r = (idx == i) ? v[i] : r;
    return r;
}

// Ascending sort of one key per lane; returns the key of sorted position `pos`.
__device__ __forceinline__ uint32_t warp_sorted_at(uint32_t x, int pos) {
    const int lane = lane_id();
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1)
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, x, stride);
            const bool asc = (lane & size) == 0, upper = (lane & stride) != 0;
            x = (asc != upper) ? min(x, o) : max(x, o);
        }
    return __shfl_sync(0xFFFFFFFFu, x, pos);
}

// Median of the n keys held by the warp (kv sorted ascending per lane, padded with
// 0xFFFFFFFF; nreal real keys in this lane).  `hint` (a key, or 0 for none) is a first pivot
// guess -- the series' median at the previous evaluation -- and need not be one of the keys.
// Returns false if a loop bound was hit.
template <int VPL>
__device__ __forceinline__ bool warp_median(const uint32_t (&kv)[VPL], const int nreal, const int n, const uint32_t hint,
                                            float &med) {
    constexpr uint32_t kNone = 0xFFFFFFFFu, kStale = 0xFFFFFFFEu;   // neither is the key of a finite value
    const int lane = lane_id();
    const bool even = !(n & 1);
    const int kq = n >> 1;             // upper middle rank (the middle for odd n)
    int lo_i = 0, hi_i = nreal;        // this lane's active run [lo_i, hi_i)
    uint32_t p = hint;
    if (p == 0u) {                     // no guess: median of the lanes' middle keys
        const unsigned have = __ballot_sync(0xFFFFFFFFu, nreal > 0);
        p = warp_sorted_at(nreal > 0 ? lane_pick<VPL>(kv, nreal >> 1) : kNone, __popc(have) >> 1);
    }
    for (int round = 0; round < 300; ++round) {
        int clt = 0, cle = 0;
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            clt += (kv[i] < p);
            cle += (kv[i] <= p);
        }
        const uint32_t tot = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)clt | ((uint32_t)cle << 16));
        const int tlt = (int)(tot & 0xFFFFu), tle = (int)(tot >> 16);   // ranks [tlt, tle) hold p
        if (kq >= tlt && kq < tle) {
            uint32_t v1 = p;
            if (even && kq == tlt)     // lower middle: the largest key below the pivot
                v1 = __reduce_max_sync(0xFFFFFFFFu, clt > 0 ? lane_pick<VPL>(kv, clt - 1) : 0u);
            med = median_from_keys(v1, p, even);
            return true;
        }
        if (kq >= tle) {
            lo_i = max(lo_i, cle);
            if (kq - tle < kWalkMax) {   // walk upwards: ranks tle, tle + 1, ...
                // rank kq - 1 when it is not reached by the walk: inside the pivot's run, or
                // (pivot not a key) the largest key below the pivot
                uint32_t v1 = p;
                if (even && kq == tle && tle == tlt)
                    v1 = __reduce_max_sync(0xFFFFFFFFu, clt > 0 ? lane_pick<VPL>(kv, clt - 1) : 0u);
                int nxt = cle, cur = tle;
                uint32_t offer = nxt < nreal ? lane_pick<VPL>(kv, nxt) : kNone;          // this lane's next key
                uint32_t after = nxt + 1 < nreal ? lane_pick<VPL>(kv, nxt + 1) : kNone;  // and the one after
                for (int step = 0; step <= kWalkMax; ++step) {
                    const uint32_t m = __reduce_min_sync(0xFFFFFFFFu, offer);
                    const bool is = (offer == m) && (m != kNone);
                    const int c = __popc(__ballot_sync(0xFFFFFFFFu, is));
                    if (c == 0) return false;
                    if (kq - 1 >= cur && kq - 1 < cur + c) v1 = m;
                    if (kq < cur + c) {
                        med = even ? median_from_keys(v1, m, true) : key2f(m);
                        return true;
                    }
                    cur += c;
                    if (is) { ++nxt; offer = after; after = kStale; }
                    if (__any_sync(0xFFFFFFFFu, offer == kStale)) {   // a lane used both prefetched keys
                        if (offer == kStale) {
                            offer = nxt < nreal ? lane_pick<VPL>(kv, nxt) : kNone;
                            after = nxt + 1 < nreal ? lane_pick<VPL>(kv, nxt + 1) : kNone;
                        }
                    }
                }
                return false;
            }
        } else {
            hi_i = min(hi_i, clt);
            if (tlt - kq <= kWalkMax) {  // walk downwards: ranks tlt - 1, tlt - 2, ...
                int nxt = clt, cur = tlt;   // this lane's next key is kv[nxt - 1]; ranks below cur are left
                uint32_t v2 = 0;
                uint32_t offer = nxt > 0 ? lane_pick<VPL>(kv, nxt - 1) : 0u;
                uint32_t after = nxt > 1 ? lane_pick<VPL>(kv, nxt - 2) : 0u;
                constexpr uint32_t kStaleLow = 1u;   // 0 and 1 are not keys of finite values either
                for (int step = 0; step <= kWalkMax + 1; ++step) {
                    const uint32_t m = __reduce_max_sync(0xFFFFFFFFu, offer);
                    const bool is = (offer == m) && (m != 0u);
                    const int c = __popc(__ballot_sync(0xFFFFFFFFu, is));
                    if (c == 0) return false;
                    // ranks [cur - c, cur) hold m
                    if (kq >= cur - c && kq < cur) v2 = m;
                    if (kq - 1 >= cur - c || (!even && kq >= cur - c)) {
                        med = even ? median_from_keys(m, v2, true) : key2f(v2);
                        return true;
                    }
                    cur -= c;
                    if (is) { --nxt; offer = after; after = kStaleLow; }
                    if (__any_sync(0xFFFFFFFFu, offer == kStaleLow)) {
                        if (offer == kStaleLow) {
                            offer = nxt > 0 ? lane_pick<VPL>(kv, nxt - 1) : 0u;
                            after = nxt > 1 ? lane_pick<VPL>(kv, nxt - 2) : 0u;
                        }
                    }
                }
                return false;
            }
        }
        // far off: next pivot is the middle key of the longest still-active run
        const uint32_t best = __reduce_max_sync(0xFFFFFFFFu, ((uint32_t)max(hi_i - lo_i, 0) << 5) | (uint32_t)lane);
        if ((best >> 5) == 0) return false;
        p = __shfl_sync(0xFFFFFFFFu, lane_pick<VPL>(kv, (lo_i + hi_i) >> 1), best & 31u);
    }
    return false;
}

// A first guess of the half-width the thread path should search around a series' smoothed
// median: 0.36 x the mean absolute deviation of the window about its median (for Gaussian
// noise that spans about +-0.29 sigma, some 3 standard errors of a 200-step median and ~22 %
// of the window).  Only a starting point: the thread path re-tunes it from its own counts.
template <int VPL>
__device__ __forceinline__ float warp_spread_guess(const uint32_t (&kv)[VPL], const int n, const float med) {
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL; ++i)
        if (kv[i] != 0xFFFFFFFFu) s += fabsf(key2f(kv[i]) - med);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    return 0.36f * s / (float)n;
}

constexpr int kThCols = 128;     // series per CTA = threads per CTA
constexpr int kThSlots = 60;     // kept keys per series
constexpr int kThTarget = 42;    // number of keys the interval is tuned to catch (windows that share few steps)
constexpr int kThRows = 8;       // rows in flight per thread
constexpr int kThMaxPasses = 12;
constexpr float kThSmooth = 0.3f;   // weight of the newest median in the interval's centre

// cnt += (x < lo); if (lo <= x <= hi) { if (addr < lim) shared[addr] = x; addr += 4; }
__device__ __forceinline__ void th_cell(const float x, const float lo, const float hi, const uint32_t lim, uint32_t &cnt,
                                        uint32_t &addr) {
    asm volatile(
        "{\n\t.reg .pred p, q, r;\n\t"
        "setp.lt.f32 p, %2, %3;\n\t"
        "setp.le.and.f32 q, %2, %4, !p;\n\t"
        "setp.lt.and.u32 r, %1, %5, q;\n\t"
        "@p add.u32 %0, %0, 1;\n\t"
        "@r st.shared.f32 [%1], %2;\n\t"
        "@q add.u32 %1, %1, 4;\n\t}"
        : "+r"(cnt), "+r"(addr)
        : "f"(x), "f"(lo), "f"(hi), "r"(lim)
        : "memory");
}
__device__ __forceinline__ uint4 th_lds4(const uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void th_sts4(const uint32_t addr, const uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Everything after the streaming pass of the one-thread-per-series path: selection among the kept
// keys (raw bits at shared-memory byte address kbase .. kaddr, clt values counted below the
// interval [klo, khi]), the update of the series' interval state, and the whole-warp fallback.
// All 32 lanes of a warp must call this together; `c` is the lane's series, `first` the ring slot
// of the window's oldest step.
template <int VPL>
__device__ __forceinline__ void th_finish(const WindowArgs &a, const int first, const int c, const bool active, const bool usable,
                                          const float hint, const float h, const uint32_t klo, const uint32_t khi,
                                          const uint32_t kbase, const uint32_t kaddr, const uint32_t clt) {
    const int n = a.n, lane = lane_id();
    const bool even = !(n & 1);
    const int k1 = (n - 1) >> 1, k2 = n >> 1;
    const int nk = (int)((kaddr - kbase) >> 2);
    bool ok = usable && (int)clt <= k1 && k2 < (int)clt + nk && nk <= kThSlots;
    const int t = k2 - (int)clt;     // rank of the upper middle among the kept keys (t >= 1 when n is even)
    float med = 0.0f;
    // ---- selection among the kept keys: the same instruction stream in every lane ---------------
    const int nkmax = (int)__reduce_max_sync(0xFFFFFFFFu, ok ? (uint32_t)nk : 0u);
    if (nkmax > 0) {
        const int nkr = (nkmax + 3) & ~3;   // <= kThSlots (a multiple of 4)
        for (int j = 0; j < nkr; j += 4) {  // raw bits -> keys; slots without a key compare above everything
            uint4 v = th_lds4(kbase + 4u * j);
            v.x = (ok && j + 0 < nk) ? key_of_bits(v.x) : 0xFFFFFFFFu;
            v.y = (ok && j + 1 < nk) ? key_of_bits(v.y) : 0xFFFFFFFFu;
            v.z = (ok && j + 2 < nk) ? key_of_bits(v.z) : 0xFFFFFFFFu;
            v.w = (ok && j + 3 < nk) ? key_of_bits(v.w) : 0xFFFFFFFFu;
            th_sts4(kbase + 4u * j, v);
        }
        // The pivot moves inside a key bracket (pl, ph) with below(pl) = al <= t - 2 and
        // below(ph) = ah >= t + 2.
        uint32_t pl = klo, ph = khi + 1u, pv = klo;
        int al = 0, ah = nk, bsave = 0;
        int done = 0;                 // 1: pv has bsave in {t - 1, t, t + 1} keys below it, 2: both ranks equal pl
        if (!ok || t <= 1) { done = 1; pv = klo; bsave = 0; }
        else if (t >= nk - 1) { done = 1; pv = khi + 1u; bsave = nk; }
        for (int pass = 0; pass < kThMaxPasses; ++pass) {
            if (__all_sync(0xFFFFFFFFu, done != 0)) break;
            if (!done) {
                if (ph - pl < 2u) {
                    done = 2;
                } else if (pass % 3 == 2) {
                    pv = pl + ((ph - pl) >> 1);
                } else {   // aim between the ends in proportion to the missing count
                    const float fr = (float)(t - al) / (float)(ah - al);
                    pv = pl + (uint32_t)((float)(ph - pl) * fr);
                    pv = pv <= pl ? pl + 1u : (pv >= ph ? ph - 1u : pv);
                }
            }
            // the loads of a third of the column are issued before their compares
            int below = 0;
#pragma unroll
            for (int j0 = 0; j0 < kThSlots / 4; j0 += 5) {
                uint4 kv4[5];
#pragma unroll
                for (int j = 0; j < 5; ++j)
                    if (4 * (j0 + j) < nkr) kv4[j] = th_lds4(kbase + 16u * (j0 + j));
#pragma unroll
                for (int j = 0; j < 5; ++j)
                    if (4 * (j0 + j) < nkr) below += (kv4[j].x < pv) + (kv4[j].y < pv) + (kv4[j].z < pv) + (kv4[j].w < pv);
            }
            if (!done) {
                if (below >= t - 1 && below <= t + 1) { done = 1; bsave = below; }
                else if (below < t) { pl = pv; al = below; }
                else { ph = pv; ah = below; }
            }
        }
        if (ok && !done) {
            if (ph - pl < 2u) done = 2; else ok = false;
        }
        // the two largest keys below the pivot (b1 >= b2), the two smallest keys not below it (u1 <= u2)
        uint32_t b1 = 0u, b2 = 0u, u1 = 0xFFFFFFFFu, u2 = 0xFFFFFFFFu;
        for (int j = 0; j < nkr; j += 4) {
            const uint4 v4 = th_lds4(kbase + 4u * j);
            const uint32_t v[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool lt = v[u] < pv;
                const uint32_t lo_v = lt ? v[u] : 0u, hi_v = lt ? 0xFFFFFFFFu : v[u];   // neutral on the other side
                b2 = max(b2, min(b1, lo_v));
                b1 = max(b1, lo_v);
                u2 = min(u2, max(u1, hi_v));
                u1 = min(u1, hi_v);
            }
        }
        uint32_t vb = b1, vu = u1;                       // bsave == t
        if (bsave == t + 1) { vb = b2; vu = b1; }
        if (bsave == t - 1) { vb = u1; vu = u2; }
        if (done == 2) { vb = pl; vu = pl; }
        if (ok) med = median_from_keys(even ? vb : vu, vu, even);
    }
    if (active && ok) {
        a.wmed[c] = med;
        if (a.wmed_user) a.wmed_user[c] = med;
        // re-tune the half-width so that the interval catches about kThTarget keys next time
        // (half of the way: one window's count is a noisy estimate of the density)
        const float f = fminf(2.0f, fmaxf(0.5f, (float)(a.target > 0 ? a.target : kThTarget) / (float)max(nk, 1)));
        a.spread[c] = h * (0.5f + 0.5f * f);
        a.centre[c] = hint + (a.smooth > 0.0f ? a.smooth : kThSmooth) * (med - hint);
    }
    // ---- series the interval did not serve: the whole warp finishes them one by one ------------
    unsigned todo = __ballot_sync(0xFFFFFFFFu, active && !ok);
    // why (diagnostic): 0 no usable interval, 1 more keys than slots, 2 median below the interval,
    // 3 above it, 4 selection did not converge
    const int why = !usable ? 0 : (nk > kThSlots ? 1 : ((int)clt > k1 ? 2 : (k2 >= (int)clt + nk ? 3 : 4)));
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const int series = __shfl_sync(0xFFFFFFFFu, c, src);
        const int why_src = __shfl_sync(0xFFFFFFFFu, why, src);
        uint32_t kv[VPL];
        int nreal = 0;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int row = lane + 32 * j;
            kv[j] = 0xFFFFFFFFu;
            if (row < n) {
                int slot = first + row;
                if (slot >= a.capacity) slot -= a.capacity;
                kv[j] = f2key(__ldg(a.ring + (size_t)slot * a.row_stride + series));
                ++nreal;
            }
        }
        lane_sort<VPL>(kv);
        float m2 = 0.0f;
        const bool ok2 = warp_median<VPL>(kv, nreal, n, 0u, m2);
        const float h0 = warp_spread_guess<VPL>(kv, n, m2);
        if (lane == 0) {
            if (!ok2) atomicOr(a.status, kStatInternal);
            a.wmed[series] = m2;
            if (a.wmed_user) a.wmed_user[series] = m2;
            a.spread[series] = h0;
            a.centre[series] = m2;
            if (a.fb_count) { atomicAdd(a.fb_count, 1u); atomicAdd(a.fb_count + 1 + why_src, 1u); }
        }
    }
}

}  // namespace guard
