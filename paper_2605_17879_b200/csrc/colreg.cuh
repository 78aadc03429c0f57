// Exact selection among keys held in the registers of a 1024-thread CTA, by histogram
// refinement on order-preserving keys: a 2048-bin shared-memory histogram over the key range
// locates the bin of the wanted rank, that bin becomes the new range, until a bin is a single
// key.
#pragma once
#include "common.cuh"

namespace guard {

constexpr int kColThreads = 1024;
constexpr int kColBins = 2048;

struct ColShared {
    uint32_t hist[kColBins];
    uint32_t warp_tot[kColThreads / 32];
    uint32_t bin, before, cnt, vmin, kmin, kmax;
    int found;
};

__device__ __forceinline__ void col_find_bin(ColShared &sh, uint32_t k) {
    constexpr int BPT = kColBins / kColThreads;
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
    if (warp == 0) {   // exclusive scan of the 32 warp totals
        const uint32_t wt = sh.warp_tot[lane];
        uint32_t wi = wt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, wi, d); if (lane >= d) wi += u; }
        sh.warp_tot[lane] = wi - wt;
    }
    __syncthreads();
    const uint32_t excl = sh.warp_tot[warp] + incl - sum;
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

// Keys of 0-based ranks k and (if want_next) k + 1 among the valid keys held in registers.
template <int VPT>
__device__ inline bool col_select_regs(const uint32_t (&key)[VPT], const uint32_t valid, uint32_t k, bool want_next,
                                ColShared &sh, uint32_t &v1, uint32_t &v2) {
    const int tid = threadIdx.x, lane = lane_id();
    // range of the keys
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll
    for (int i = 0; i < VPT; ++i)
        if ((valid >> i) & 1u) { kmin = min(kmin, key[i]); kmax = max(kmax, key[i]); }
    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
    if (tid == 0) { sh.kmin = 0xFFFFFFFFu; sh.kmax = 0u; }
    __syncthreads();
    if (lane == 0) { atomicMin(&sh.kmin, kmin); atomicMax(&sh.kmax, kmax); }
    __syncthreads();
    uint32_t base = sh.kmin, width = sh.kmax - sh.kmin;
    uint32_t krem = k, ceq = 0;
    v1 = 0;
    for (;;) {
        const int bits = 32 - __clz(width);
        const int shv = bits > 11 ? bits - 11 : 0;
        for (int i = tid; i < kColBins; i += kColThreads) sh.hist[i] = 0;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const uint32_t off = key[i] - base;
            if (((valid >> i) & 1u) && off <= width) atomicAdd(&sh.hist[off >> shv], 1u);
        }
        __syncthreads();
        col_find_bin(sh, krem);
        if (!sh.found) return false;
        krem -= sh.before;
        if (shv == 0) { v1 = base + sh.bin; ceq = sh.cnt; break; }
        base += sh.bin << shv;
        width = (1u << shv) - 1u;
        __syncthreads();
    }
    v2 = v1;
    if (want_next && krem + 1 >= ceq) {   // next order statistic: the smallest key above v1
        if (tid == 0) sh.vmin = 0xFFFFFFFFu;
        __syncthreads();
        uint32_t c = 0xFFFFFFFFu;
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            if (((valid >> i) & 1u) && key[i] > v1) c = min(c, key[i]);
        c = __reduce_min_sync(0xFFFFFFFFu, c);
        if (lane == 0 && c != 0xFFFFFFFFu) atomicMin(&sh.vmin, c);
        __syncthreads();
        v2 = sh.vmin;
        if (v2 == 0xFFFFFFFFu) return false;
    }
    __syncthreads();
    return true;
}

}  // namespace guard
