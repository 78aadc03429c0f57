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

// ---- hinted selection ---------------------------------------------------------------------------
// When the caller can bracket the wanted order statistic (the previous result of the same call site:
// consecutive steps of a fleet have almost the same cross-rank median and MAD), two cluster barriers
// settle it: (1) every CTA counts its keys below the bracket [blo, bhi] and bins those inside
// (2048 bins over the bracket); the summed histograms give the bins of ranks k and k + 1 and prove
// from the counts that the bracket holds them; (2) the few keys of those bins are gathered from all
// CTAs and ranked directly.  Anything else (the counts do not prove the bracket, more gathered keys
// than the lists hold) returns false and the caller runs the range-refining selection above.
constexpr int kHintList = 64;     // gathered keys per CTA
constexpr int kHintAll = 256;     // gathered keys per cluster

struct HintShared {
    uint32_t hist[2][kColBins];   // one buffer per selection of a launch (median, MAD): no reuse, no barrier in between
    uint32_t below[2], nlist[2];
    uint32_t list[2][kHintList];
    uint32_t all[kHintAll];
    uint32_t warp_tot[kColThreads / 32];
    uint32_t bin[2], before[2], total;
    uint32_t res[2];
    int found[2];
};

// Zeroes the buffers of both selections (call once, then __syncthreads or a cluster barrier).
__device__ __forceinline__ void hint_clear(HintShared &hs) {
    const int tid = threadIdx.x;
    for (int i = tid; i < 2 * kColBins; i += kColThreads) (&hs.hist[0][0])[i] = 0;
    if (tid < 2) { hs.below[tid] = 0; hs.nlist[tid] = 0; }
}

// Bins of ranks r1 and r2 in the histogram summed over the cluster, and its total.
template <int NC>
__device__ __forceinline__ void hint_find_two(HintShared &hs, const int which, const uint32_t r1, const uint32_t r2) {
    constexpr int BPT = kColBins / kColThreads;
    const int tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    uint32_t loc[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        loc[i] = 0;
#pragma unroll
        for (int c = 0; c < NC; ++c) loc[i] += cl_ld(cl_addr(&hs.hist[which][tid * BPT + i], (uint32_t)c));
        sum += loc[i];
    }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
    if (lane == 31) hs.warp_tot[warp] = incl;
    if (tid < 2) hs.found[tid] = 0;
    __syncthreads();
    if (warp == 0) {   // exclusive scan of the 32 warp totals
        const uint32_t wt = hs.warp_tot[lane];
        uint32_t wi = wt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, wi, d); if (lane >= d) wi += u; }
        hs.warp_tot[lane] = wi - wt;
        if (lane == 31) hs.total = wi;
    }
    __syncthreads();
    const uint32_t excl = hs.warp_tot[warp] + incl - sum;
    uint32_t run = excl;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        if (r1 >= run && r1 < run + loc[i]) { hs.bin[0] = (uint32_t)(tid * BPT + i); hs.before[0] = run; hs.found[0] = 1; }
        if (r2 >= run && r2 < run + loc[i]) { hs.bin[1] = (uint32_t)(tid * BPT + i); hs.before[1] = run; hs.found[1] = 1; }
        run += loc[i];
    }
    __syncthreads();
}

// Keys of ranks k and (if want_next) k + 1, given a bracket.  `which` picks the buffer set (each set is used by
// one selection per launch).  n_in returns the number of keys inside the bracket (for tuning its width).
// All threads of all CTAs of the cluster call this together and get the same answer.
template <int VPT, int NC>
__device__ inline bool colc_select_hinted(const uint32_t (&key)[VPT], const uint32_t valid, const uint32_t k,
                                          const bool want_next, const uint32_t blo, const uint32_t bhi, HintShared &hs,
                                          const int which, uint32_t &v1, uint32_t &v2, uint32_t &n_in, int &side) {
    const int tid = threadIdx.x, lane = lane_id();
    const uint32_t width = bhi - blo;
    const int bits = 32 - __clz(width);
    const int shv = bits > 11 ? bits - 11 : 0;
    uint32_t below = 0;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const bool v = (valid >> i) & 1u;
        const uint32_t off = key[i] - blo;
        below += (v && key[i] < blo) ? 1u : 0u;
        if (v && key[i] >= blo && off <= width) atomicAdd(&hs.hist[which][off >> shv], 1u);
    }
    below = __reduce_add_sync(0xFFFFFFFFu, below);
    if (lane == 0 && below) atomicAdd(&hs.below[which], below);
    cl_sync();   // (1) counts and histograms of every CTA are complete
    uint32_t tb = 0;
#pragma unroll
    for (int c = 0; c < NC; ++c) tb += cl_ld(cl_addr(&hs.below[which], (uint32_t)c));
    n_in = 0;
    side = 0;
    if (tb > k) { side = -1; return false; }              // the wanted rank lies below the bracket
    const uint32_t r1 = k - tb, r2 = want_next ? r1 + 1 : r1;
    hint_find_two<NC>(hs, which, r1, r2);
    n_in = hs.total;
    if (!hs.found[0] || !hs.found[1]) { side = 1; return false; }   // ... or above it
    const uint32_t b1 = hs.bin[0], b2 = hs.bin[1];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const uint32_t off = key[i] - blo;
        if (((valid >> i) & 1u) && key[i] >= blo && off <= width) {
            const uint32_t b = off >> shv;
            if (b == b1 || b == b2) {
                const uint32_t pos = atomicAdd(&hs.nlist[which], 1u);
                if (pos < (uint32_t)kHintList) hs.list[which][pos] = key[i];
            }
        }
    }
    cl_sync();   // (2) the gathered keys of every CTA are complete
    uint32_t cnt[NC], T = 0;
    bool fits = true;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        cnt[c] = cl_ld(cl_addr(&hs.nlist[which], (uint32_t)c));
        fits = fits && cnt[c] <= (uint32_t)kHintList;
        T += cnt[c];
    }
    if (!fits || T > (uint32_t)kHintAll) return false;    // ties beyond the lists: the general selection handles them
    if ((uint32_t)tid < T) {
        uint32_t t = (uint32_t)tid, val = 0;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            if (t < cnt[c]) { val = cl_ld(cl_addr(&hs.list[which][t], (uint32_t)c)); t = 0xFFFFFFFFu; }
            else if (t != 0xFFFFFFFFu) t -= cnt[c];
        }
        hs.all[tid] = val;
    }
    __syncthreads();
    const uint32_t q1 = r1 - hs.before[0];   // rank inside the gathered keys (bins b1 <= b2 with nothing in between)
    if ((uint32_t)tid < T) {
        const uint32_t mine = hs.all[tid];
        uint32_t rk = 0;
        for (uint32_t j = 0; j < T; ++j) {
            const uint32_t o = hs.all[j];
            rk += (o < mine || (o == mine && j < (uint32_t)tid)) ? 1u : 0u;
        }
        if (rk == q1) hs.res[0] = mine;
        if (rk == q1 + 1) hs.res[1] = mine;
    }
    __syncthreads();
    v1 = hs.res[0];
    v2 = want_next ? hs.res[1] : v1;
    const bool ok = q1 + (want_next ? 1u : 0u) < T;
    __syncthreads();   // res / all may be rewritten by the next selection
    return ok;
}

}  // namespace guard
