// Direct cross-rank selection of one row: 8-bit most-significant-digit radix select on
// order-preserving keys with one 256-bin shared-memory histogram per metric; lanes that hit
// the same bin are merged with __match_any_sync before the shared-memory atomic.  Used by
// the direct kernel (small fleets, metric counts the fast paths do not cover, the sweep's
// percentile cut) and, inline, by the fast paths when a sampled interval fails.
#pragma once
#include "kernels.h"

namespace guard {

struct XrShared {
    uint32_t prefix[kMaxMetrics];  // key digits decided so far
    uint32_t krem[kMaxMetrics];    // rank still to find inside the current prefix
    uint32_t ceq[kMaxMetrics];     // copies of the selected key
    uint32_t v2[kMaxMetrics];      // next order statistic (key)
    uint32_t k1[kMaxMetrics];      // wanted 0-based rank
    int need_above[kMaxMetrics];
    float med[kMaxMetrics];
    float rhs[kMaxMetrics];
    int any_need;
};

// Finds the bin of a 256-bin histogram that holds 0-based rank k.  All 32 lanes call it.
__device__ __forceinline__ void warp_find_bin(const uint32_t *h, uint32_t k, int &bin, uint32_t &before,
                                              uint32_t &cnt, bool &ok) {
    const int lane = lane_id();
    uint32_t loc[8];
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        loc[i] = h[lane * 8 + i];
        sum += loc[i];
    }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += t;
    }
    uint32_t excl = incl - sum;
    bool mine = (k >= excl) && (k < incl);
    unsigned ball = __ballot_sync(0xFFFFFFFFu, mine);
    ok = ball != 0;
    int src = ok ? (__ffs(ball) - 1) : 31;
    int b = 7;
    uint32_t bef = excl, c = 0;
    if (lane == src) {
        uint32_t run = excl;
        b = 7;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (k >= run && k < run + loc[i]) { b = i; bef = run; c = loc[i]; }
            run += loc[i];
        }
    }
    bin = __shfl_sync(0xFFFFFFFFu, lane * 8 + b, src);
    before = __shfl_sync(0xFFFFFFFFu, bef, src);
    cnt = __shfl_sync(0xFFFFFFFFu, c, src);
}

// CTA-wide radix select over the columns of one row.  For every metric m finds the key
// of 0-based rank sh.k1[m] (into sh.prefix[m]) and, if want_next, the key of the next
// rank (into sh.v2[m]).  keyf(x, m) maps a value to its key.
template <class KeyFn>
__device__ inline void cta_select(const float *__restrict__ row, int R, int M, bool want_next, KeyFn keyf,
                           uint32_t *hist, XrShared &sh, uint32_t *status) {
    const int tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    const int nwarps = blockDim.x >> 5;
    for (int i = tid; i < M * 256; i += blockDim.x) hist[i] = 0;
    if (tid < M) {
        sh.prefix[tid] = 0;
        sh.krem[tid] = sh.k1[tid];
    }
    __syncthreads();
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int r0 = 0; r0 < R; r0 += blockDim.x) {
            const int r = r0 + tid;
            const bool in = r < R;
            for (int m = 0; m < M; ++m) {
                bool valid = in;
                uint32_t key = 0;
                if (in) {
                    key = keyf(row[(size_t)r * M + m], m);
                    if (pass > 0) valid = ((key ^ sh.prefix[m]) >> (shift + 8)) == 0;
                }
                const uint32_t digit = (key >> shift) & 255u;
                const uint32_t tag = valid ? digit : (256u + lane);
                const unsigned peers = __match_any_sync(0xFFFFFFFFu, tag);
                if (valid && lane == __ffs(peers) - 1) atomicAdd(&hist[m * 256 + digit], __popc(peers));
            }
        }
        __syncthreads();
        for (int m = warp; m < M; m += nwarps) {
            int bin;
            uint32_t before, cnt;
            bool ok;
            warp_find_bin(hist + m * 256, sh.krem[m], bin, before, cnt, ok);
            __syncwarp();
            for (int i = lane; i < 256; i += 32) hist[m * 256 + i] = 0;
            if (lane == 0) {
                if (!ok && status) atomicOr(status, kStatInternal);
                sh.prefix[m] |= (uint32_t)bin << shift;
                sh.krem[m] -= before;
                sh.ceq[m] = cnt;
            }
        }
        __syncthreads();
    }
    if (!want_next) return;
    // The next order statistic equals the selected key if further copies of it remain,
    // otherwise it is the smallest key above it.
    if (tid == 0) sh.any_need = 0;
    __syncthreads();
    if (tid < M) {
        const int need = (sh.krem[tid] + 1 >= sh.ceq[tid]);
        sh.need_above[tid] = need;
        sh.v2[tid] = need ? 0xFFFFFFFFu : sh.prefix[tid];
        if (need) sh.any_need = 1;
    }
    __syncthreads();
    if (sh.any_need) {
        for (int r0 = 0; r0 < R; r0 += blockDim.x) {
            const int r = r0 + tid;
            for (int m = 0; m < M; ++m) {
                if (!sh.need_above[m]) continue;
                uint32_t cand = 0xFFFFFFFFu;
                if (r < R) {
                    const uint32_t key = keyf(row[(size_t)r * M + m], m);
                    if (key > sh.prefix[m]) cand = key;
                }
                cand = __reduce_min_sync(0xFFFFFFFFu, cand);
                if (lane == 0 && cand != 0xFFFFFFFFu) atomicMin(&sh.v2[m], cand);
            }
        }
    }
    __syncthreads();
}

template <typename MaskT>
__device__ inline void write_exceedance(const float *__restrict__ row, int R, int M, const MetricParams &p,
                                 const XrShared &sh, MaskT *out) {
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        uint32_t mask = 0;
        for (int m = 0; m < M; ++m)
            if (exceeds(row[(size_t)r * M + m], sh.med[m], p.dir[m], sh.rhs[m])) mask |= 1u << m;
        out[r] = (MaskT)mask;
    }
}

// All threads of the CTA: median, MAD (and optional extra order statistic) of every column of
// row s of the launch, plus the exceedance mask of the row.  hist: M * 256 words of shared
// memory.
__device__ inline void xrank_direct_step(const XrankArgs &a, const MetricParams &p, const int s, uint32_t *hist,
                                         XrShared &sh) {
    const int tid = threadIdx.x;
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + s) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const bool even = (R & 1) == 0;

    if (a.check_finite) {
        bool bad = false;
        for (size_t i = tid; i < (size_t)R * M; i += blockDim.x) bad |= nonfinite_bits(__float_as_uint(row[i]));
        if (__any_sync(0xFFFFFFFFu, bad) && lane_id() == 0) atomicOr(a.status, kStatNonFinite);
    }
    // median of every column
    if (tid < M) sh.k1[tid] = (uint32_t)((R - 1) / 2);
    __syncthreads();
    cta_select(row, R, M, even, [](float x, int) { return f2key(x); }, hist, sh, a.status);
    if (tid < M) {
        const float med = median_from_keys(sh.prefix[tid], even ? sh.v2[tid] : sh.prefix[tid], even);
        sh.med[tid] = med;
        a.med[(size_t)s * M + tid] = med;
        if (a.med_user) a.med_user[(size_t)s * M + tid] = med;
    }
    __syncthreads();
    // median of the absolute deviations about it
    const float *medp = sh.med;
    cta_select(row, R, M, even, [medp](float x, int m) { return f2key(fabsf(__fsub_rn(x, medp[m]))); }, hist, sh,
               a.status);
    if (tid < M) {
        const float mad = median_from_keys(sh.prefix[tid], even ? sh.v2[tid] : sh.prefix[tid], even);
        a.mad[(size_t)s * M + tid] = mad;
        if (a.mad_user) a.mad_user[(size_t)s * M + tid] = mad;
        const float sc = scale_of(mad, sh.med[tid], p.floor_rel[tid], p.floor_abs[tid]);
        sh.rhs[tid] = __fmul_rn(p.thrp[tid], sc);
    }
    __syncthreads();
    if (a.mask_base) {
        if (a.mask_bytes == 1)
            write_exceedance<uint8_t>(row, R, M, p, sh, (uint8_t *)a.mask_base + (size_t)slot * R);
        else
            write_exceedance<uint32_t>(row, R, M, p, sh, (uint32_t *)a.mask_base + (size_t)slot * R);
    }
    if (a.cut) {
        __syncthreads();
        if (tid < M) sh.k1[tid] = (uint32_t)a.cut_rank[tid];
        __syncthreads();
        cta_select(row, R, M, false, [](float x, int) { return f2key(x); }, hist, sh, a.status);
        if (tid < M) a.cut[(size_t)s * M + tid] = key2f(sh.prefix[tid]);
    }
}

}  // namespace guard
