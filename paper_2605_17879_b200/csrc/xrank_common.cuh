// Helpers shared by the fast cross-rank paths.
#pragma once
#include <math_constants.h>

#include "common.cuh"

namespace guard {

// previous / next float32 in the total order (used to open sampled intervals by one ulp)
__device__ __forceinline__ float fdown(float x) { return __uint_as_float(f2key(x) == 0 ? __float_as_uint(x) : bits_of_key(f2key(x) - 1)); }
__device__ __forceinline__ float fup(float x) { return __uint_as_float(bits_of_key(f2key(x) + 1)); }

// Ascending bitonic sort of 32 * EPL keys held EPL per lane (element e lives in lane e / EPL,
// register e % EPL): small strides are register-to-register, large ones go over shuffles.
// The stage loops are kept rolled (only the per-register loop is unrolled): the network runs
// once per CTA, and fully unrolled it is tens of kilobytes of straight-line code whose
// instruction-cache misses cost more than the sort itself.
template <int EPL, int STRIDE>
__device__ __forceinline__ void bitonic_in_lane(uint32_t (&v)[EPL], const int lane, const int size) {
#pragma unroll
    for (int j = 0; j < EPL; ++j) {
        if ((j & STRIDE) == 0) {
            const bool asc = (((lane * EPL + j) & size) == 0);
            const uint32_t x = v[j], y = v[j | STRIDE];
            const uint32_t mn = min(x, y), mx = max(x, y);
            v[j] = asc ? mn : mx;
            v[j | STRIDE] = asc ? mx : mn;
        }
    }
}

template <int EPL>
__device__ __forceinline__ void warp_bitonic_sort(uint32_t (&v)[EPL], const int lane) {
    constexpr int N = 32 * EPL;
#pragma unroll 1
    for (int size = 2; size <= N; size <<= 1) {
#pragma unroll 1
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            if (stride >= EPL) {   // partner element lives in lane ^ (stride / EPL), same register
                const int lm = stride / EPL;
                const bool upper = (lane & lm) != 0;
#pragma unroll
                for (int j = 0; j < EPL; ++j) {
                    const bool asc = (((lane * EPL + j) & size) == 0);
                    const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, v[j], lm);
                    v[j] = (asc != upper) ? min(v[j], o) : max(v[j], o);
                }
            } else {               // both elements in this lane
                switch (stride) {
                    case 1: bitonic_in_lane<EPL, 1>(v, lane, size); break;
                    case 2: if (EPL > 2) bitonic_in_lane<EPL, (EPL > 2 ? 2 : 1)>(v, lane, size); break;
                    case 4: if (EPL > 4) bitonic_in_lane<EPL, (EPL > 4 ? 4 : 1)>(v, lane, size); break;
                    case 8: if (EPL > 8) bitonic_in_lane<EPL, (EPL > 8 ? 8 : 1)>(v, lane, size); break;
                    case 16: if (EPL > 16) bitonic_in_lane<EPL, (EPL > 16 ? 16 : 1)>(v, lane, size); break;
                    default: break;
                }
            }
        }
    }
}

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

}  // namespace guard
