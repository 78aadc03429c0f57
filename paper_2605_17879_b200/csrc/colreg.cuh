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

// ---- the same selection with one column spread over a cluster of NC CTAs ------------------------
// Every CTA holds a share of the column in registers and builds a histogram of its own; the CTAs
// read one another's histograms through distributed shared memory and each scans the sum, so all of
// them find the same bin without any further exchange.  Control flow is the same in every CTA of
// the cluster (it depends only on the summed histograms), so the cluster barriers always meet.
__device__ __forceinline__ uint32_t cl_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cl_addr(const void *p, uint32_t rank) {   // address of p in CTA `rank` of the cluster
    uint32_t o;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(o) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(rank));
    return o;
}
__device__ __forceinline__ uint32_t cl_ld(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void cl_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int NC>
__device__ __forceinline__ void colc_find_bin(ColShared &sh, uint32_t k) {
    constexpr int BPT = kColBins / kColThreads;
    const int tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    uint32_t loc[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        loc[i] = 0;
#pragma unroll
        for (int c = 0; c < NC; ++c) loc[i] += cl_ld(cl_addr(&sh.hist[tid * BPT + i], (uint32_t)c));
        sum += loc[i];
    }
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

// Keys of 0-based ranks k and (if want_next) k + 1 among the valid keys held in the registers of the
// NC CTAs of the cluster.  All threads of all CTAs call this together and get the same answer.
template <int VPT, int NC>
__device__ inline bool colc_select_regs(const uint32_t (&key)[VPT], const uint32_t valid, uint32_t k, bool want_next,
                                        ColShared &sh, uint32_t &v1, uint32_t &v2) {
    const int tid = threadIdx.x, lane = lane_id();
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll
    for (int i = 0; i < VPT; ++i)
        if ((valid >> i) & 1u) { kmin = min(kmin, key[i]); kmax = max(kmax, key[i]); }
    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
    if (tid == 0) { sh.kmin = 0xFFFFFFFFu; sh.kmax = 0u; }
    __syncthreads();
    if (lane == 0) { atomicMin(&sh.kmin, kmin); atomicMax(&sh.kmax, kmax); }
    cl_sync();   // every CTA's range is final
    uint32_t base = 0xFFFFFFFFu, top = 0u;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        base = min(base, cl_ld(cl_addr(&sh.kmin, (uint32_t)c)));
        top = max(top, cl_ld(cl_addr(&sh.kmax, (uint32_t)c)));
    }
    uint32_t width = top - base;
    uint32_t krem = k, ceq = 0;
    v1 = 0;
    bool ok = true;
    for (;;) {
        const int bits = 32 - __clz(width);
        const int shv = bits > 11 ? bits - 11 : 0;
        cl_sync();   // nobody reads this CTA's histogram (or range) any more
        for (int i = tid; i < kColBins; i += kColThreads) sh.hist[i] = 0;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const uint32_t off = key[i] - base;
            if (((valid >> i) & 1u) && off <= width) atomicAdd(&sh.hist[off >> shv], 1u);
        }
        cl_sync();   // all histograms are complete
        colc_find_bin<NC>(sh, krem);
        if (!sh.found) { ok = false; break; }
        krem -= sh.before;
        if (shv == 0) { v1 = base + sh.bin; ceq = sh.cnt; break; }
        base += sh.bin << shv;
        width = (1u << shv) - 1u;
    }
    v2 = v1;
    const bool need_next = ok && want_next && krem + 1 >= ceq;   // the same in every CTA
    cl_sync();       // histograms are no longer read
    if (need_next) { // next order statistic: the smallest key above v1, over the whole cluster
        if (tid == 0) sh.vmin = 0xFFFFFFFFu;
        __syncthreads();
        uint32_t c = 0xFFFFFFFFu;
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            if (((valid >> i) & 1u) && key[i] > v1) c = min(c, key[i]);
        c = __reduce_min_sync(0xFFFFFFFFu, c);
        if (lane == 0 && c != 0xFFFFFFFFu) atomicMin(&sh.vmin, c);
        cl_sync();
        v2 = 0xFFFFFFFFu;
#pragma unroll
        for (int cc = 0; cc < NC; ++cc) v2 = min(v2, cl_ld(cl_addr(&sh.vmin, (uint32_t)cc)));
        if (v2 == 0xFFFFFFFFu) ok = false;
        cl_sync();   // vmin has been read everywhere before it is reused
    }
    return ok;
}

}  // namespace guard
