// Exact selection inside one warp: the keys of a series live in the registers of the warp's lanes
// (VPL per lane).  Shared by the window kernels (window.cu) and the node sweep (sweep.cu).
#pragma once
#include "common.cuh"

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

}  // namespace guard
