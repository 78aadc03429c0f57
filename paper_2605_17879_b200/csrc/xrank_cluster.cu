// Cross-rank selection, cluster path: one thread-block CLUSTER of four 256-thread CTAs per
// step, for fleets of a few thousand ranks and more with 4 or 8 metrics.  Each CTA sweeps a
// quarter of the step's ranks; the four CTAs exchange interval ends, counts and results
// through distributed shared memory, and every CTA owns the selections of M / 4 metrics.
// Small CTAs (some 30 KB of shared memory) let five or six of them share an SM, so that the
// selection phase of one step overlaps the sweeps of others and a launch of a few hundred
// steps fills all SMs evenly.
//
//   0. sample   (owner CTA of a metric) 32 spread values are sorted in a warp; their median
//               and quartile span fix a linear map onto 2048 bins; every stride-th rank of
//               the column (about 4096 values) is counted into those bins; the bins that
//               hold the sample ranks middle +- delta and quartiles +- delta_q give the
//               interval [lo, hi] of the column's median and [dlo, dhi] of its MAD;
//   1. sweep    every CTA counts its elements below lo and keeps those inside [lo, hi] in a
//               list in its own shared memory (one reservation per warp and batch);
//   2. select   the owner checks from the summed counts that the interval holds the middle
//               ranks and finds them among the four kept lists (read through distributed
//               shared memory) by histogram refinement on order-preserving keys;
//   3. sweep    the same for |x - med| in [dlo, dhi]; elements that might exceed the
//               threshold are rare: those clear of the threshold's possible range set their
//               exceedance bit at once, the others are deferred;
//   4. select   exact MAD, threshold; 5. the deferred elements are settled.
//
// Intervals only steer the work: the counts prove that an interval holds what it should, a
// missed interval is moved by its own width once, and if that fails too (or a list
// overflows) the first CTA of the cluster recomputes the step with the direct radix select.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "xrank_common.cuh"
#include "xrank_direct.cuh"

namespace cg = cooperative_groups;

namespace guard {

namespace {

constexpr int kClP = 4;            // CTAs per cluster
constexpr int kClThreads = 256;
constexpr int kClU = 4;            // ranks per thread and sweep batch
constexpr int kClAmb = 256;        // deferred exceedance decisions per CTA
constexpr int kClSlack = 128;      // words behind each kept list that absorb the stores of a full list
constexpr int kClSample = 4096;    // target number of sampled ranks per column
constexpr int kClSBins = 2048;     // sample histogram bins (16-bit counters, two per word)
constexpr int kClBins = 1024;      // selection histogram bins
constexpr int kClMaxM = 8;
constexpr float kFltMax = 3.402823466e+38f;

struct ClGeom {
    int slice;      // ranks per CTA (a multiple of 16)
    int cap;        // kept elements per metric and CTA
    int stride;     // sampled ranks are stride / 2, stride / 2 + stride, ...
    int s;          // number of sampled ranks
    int delta;      // half-width of the median interval in sample ranks
    int delta_q;    // half-width of the quartile intervals in sample ranks
};

struct ClSel {      // per selection group
    uint32_t warp_tot[8];
    uint32_t bin, before, cnt, vmin;
    int found;
    float inv_bw, off;
    int sample_ok;
    uint32_t scount, r1, r2;
    uint32_t small[32];
    uint32_t tk[6], tb[6];
};

struct ClShared {
    float lo[kClMaxM], hi[kClMaxM], dlo[kClMaxM], dhi[kClMaxM];
    float med[kClMaxM], rlo[kClMaxM], rhi[kClMaxM], rhs[kClMaxM];
    float sgn[kClMaxM];               // +1 / -1: the metric's bad direction
    uint32_t cnt[kClMaxM];            // elements below the interval (summed over the cluster at the owner)
    uint32_t n32[4];                  // this CTA's kept counts, two 16-bit fields per word (metric m: word m / 2)
    uint32_t namb;
    int fail;                         // 1 = an interval missed (sweep again), 2 = give up
    ClSel sel[2];
};

// Named barrier of one selection group (ids 1 and 2: literal ids keep the other barriers free).
__device__ __forceinline__ void cl_group_bar(int id, int nthreads) {
    if (id == 1) asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
    else asm volatile("bar.sync 2, %0;" ::"r"(nthreads) : "memory");
}

// Distributed shared memory: the address of one of this CTA's shared variables in CTA `rank`
// of the cluster (a 32-bit shared::cluster address), and accesses through such addresses.
__device__ __forceinline__ uint32_t cl_map(const void *p, int rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(rank));
    return out;
}
__device__ __forceinline__ uint32_t cl_ld(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void cl_st(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cl_stf(uint32_t addr, float v) { cl_st(addr, __float_as_uint(v)); }
__device__ __forceinline__ void cl_red_add(uint32_t addr, uint32_t v) {
    asm volatile("red.shared::cluster.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cl_red_max(uint32_t addr, int v) {
    asm volatile("red.shared::cluster.max.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cl_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Ascending sort of one key per lane (bitonic network over shuffles).
__device__ __forceinline__ uint32_t cl_warp_sort(uint32_t x, const int lane) {
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

// The kept lists of one metric in the four CTAs of the cluster.
struct ClSegs {
    uint32_t p[kClP];   // shared::cluster addresses
    uint32_t n[kClP];
};

// Finds the bin of hist[kClBins] holding 0-based rank k (the G threads of one group).
template <int G>
__device__ __forceinline__ void cl_find_bin(const uint32_t *hist, ClSel &gs, uint32_t k, int gt, int barid) {
    constexpr int BPT = kClBins / G;
    const int lane = gt & 31, gw = gt >> 5;
    uint32_t loc[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) { loc[i] = hist[gt * BPT + i]; sum += loc[i]; }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += u; }
    if (lane == 31) gs.warp_tot[gw] = incl;
    if (gt == 0) gs.found = 0;
    cl_group_bar(barid, G);
    uint32_t off = 0;
    for (int w = 0; w < gw; ++w) off += gs.warp_tot[w];
    const uint32_t excl = off + incl - sum;
    if (k >= excl && k < excl + sum) {
        uint32_t run = excl;
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            if (k >= run && k < run + loc[i]) { gs.bin = (uint32_t)(gt * BPT + i); gs.before = run; gs.cnt = loc[i]; gs.found = 1; }
            run += loc[i];
        }
    }
    cl_group_bar(barid, G);
}

// Keys of ranks k and (if want_next) k + 1 among the kept elements (raw float bits), all of
// whose keys lie in [base, base + width].  Called by the G threads of a group.
template <int G>
__device__ bool cl_select(const ClSegs &sg, uint32_t k, bool want_next, uint32_t base, uint32_t width, uint32_t *hist,
                          ClSel &gs, int gt, int barid, uint32_t &v1, uint32_t &v2) {
    uint32_t krem = k, ceq = 0;
    bool ok = true;
    v1 = 0;
    for (;;) {
        const int bits = 32 - __clz(width);
        const int shv = bits > 10 ? bits - 10 : 0;
        for (int i = gt; i < kClBins; i += G) hist[i] = 0;
        cl_group_bar(barid, G);
#pragma unroll
        for (int c = 0; c < kClP; ++c) {
            const uint32_t lp = sg.p[c];
            const uint32_t n = sg.n[c];
            for (uint32_t i = gt; i < n; i += G) {
                const uint32_t off = key_of_bits(cl_ld(lp + 4u * i)) - base;
                if (off <= width) atomicAdd(&hist[off >> shv], 1u);
            }
        }
        cl_group_bar(barid, G);
        cl_find_bin<G>(hist, gs, krem, gt, barid);
        if (!gs.found) { ok = false; break; }
        krem -= gs.before;
        if (shv == 0) { v1 = base + gs.bin; ceq = gs.cnt; break; }
        base += gs.bin << shv;
        width = (1u << shv) - 1u;
        cl_group_bar(barid, G);
    }
    v2 = v1;
    if (ok && want_next && krem + 1 >= ceq) {   // next order statistic: smallest key above v1
        if (gt == 0) gs.vmin = 0xFFFFFFFFu;
        cl_group_bar(barid, G);
        uint32_t cm = 0xFFFFFFFFu;
#pragma unroll
        for (int c = 0; c < kClP; ++c) {
            const uint32_t lp = sg.p[c];
            const uint32_t n = sg.n[c];
            for (uint32_t i = gt; i < n; i += G) {
                const uint32_t key = key_of_bits(cl_ld(lp + 4u * i));
                if (key > v1) cm = min(cm, key);
            }
        }
        cm = __reduce_min_sync(0xFFFFFFFFu, cm);
        if ((gt & 31) == 0 && cm != 0xFFFFFFFFu) atomicMin(&gs.vmin, cm);
        cl_group_bar(barid, G);
        v2 = gs.vmin;
        if (v2 == 0xFFFFFFFFu) ok = false;
    }
    cl_group_bar(barid, G);
    return ok;
}

// The same selection with the kept elements of the four lists held in registers (at most
// JMAX per list and thread), fetched with one batch of distributed-shared-memory loads.  A
// 1024-bin histogram over the interval locates the bin of rank k; while that bin holds more
// than 32 keys it becomes the next, narrower range; then the bin's keys are gathered and one
// warp ranks them.  The next order statistic is the following gathered key or, if the bin ends
// there, the smallest key above the bin.
template <int G, int JMAX>
__device__ bool cl_select_regs(const ClSegs &sg, uint32_t k, bool want_next, uint32_t base, uint32_t width, uint32_t *hist,
                               ClSel &gs, int gt, int barid, uint32_t &v1, uint32_t &v2) {
    uint32_t off[kClP * JMAX];   // key - base; 0xFFFFFFFF (beyond any width) where there is no element
#pragma unroll
    for (int c = 0; c < kClP; ++c)
#pragma unroll
        for (int j = 0; j < JMAX; ++j) {
            const uint32_t i = (uint32_t)(gt + j * G);
            off[c * JMAX + j] = 0x7F800000u;   // bits of +inf: its key lies above every finite key
            if (i < sg.n[c]) off[c * JMAX + j] = cl_ld(sg.p[c] + 4u * i);
        }
#pragma unroll
    for (int e = 0; e < kClP * JMAX; ++e) {
        const uint32_t key = key_of_bits(off[e]);
        off[e] = key >= base ? key - base : 0xFFFFFFFFu;
    }
    uint32_t krem = k;
    bool ok = true;
    v1 = v2 = 0;
    for (int round = 0; round < 4; ++round) {
        const int bits = 32 - __clz(width);
        const int shv = bits > 10 ? bits - 10 : 0;
        for (int i = gt; i < kClBins; i += G) hist[i] = 0;
        if (gt == 0) { gs.scount = 0; gs.vmin = 0xFFFFFFFFu; }
        cl_group_bar(barid, G);
#pragma unroll
        for (int e = 0; e < kClP * JMAX; ++e)
            if (off[e] <= width) atomicAdd(&hist[off[e] >> shv], 1u);
        cl_group_bar(barid, G);
        cl_find_bin<G>(hist, gs, krem, gt, barid);
        if (!gs.found) { ok = false; break; }
        krem -= gs.before;
        const uint32_t bin = gs.bin, cnt = gs.cnt;
        if (cnt <= 32u || shv == 0) {
            if (shv == 0) {   // the bin is a single key
                v1 = base + bin;
                v2 = v1;
                if (!(want_next && krem + 1 >= cnt)) break;
            }
            // gather the bin's keys, and the smallest key above the bin
            uint32_t mn = 0xFFFFFFFFu;
#pragma unroll
            for (int e = 0; e < kClP * JMAX; ++e) {
                if (off[e] <= width) {
                    const uint32_t b = off[e] >> shv;
                    if (b == bin && shv != 0) {
                        const uint32_t pos = atomicAdd(&gs.scount, 1u);
                        if (pos < 32u) gs.small[pos] = off[e];
                    } else if (b > bin) {
                        mn = min(mn, off[e]);
                    }
                }
            }
            mn = __reduce_min_sync(0xFFFFFFFFu, mn);
            if ((gt & 31) == 0 && mn != 0xFFFFFFFFu) atomicMin(&gs.vmin, mn);
            cl_group_bar(barid, G);
            if (shv == 0) {
                v2 = gs.vmin == 0xFFFFFFFFu ? 0xFFFFFFFFu : base + gs.vmin;
                if (gs.vmin == 0xFFFFFFFFu) ok = false;
                break;
            }
            if (gt < 32) {   // rank the gathered keys (ties by position): ranks krem and krem + 1
                const uint32_t mine = (uint32_t)gt < cnt ? gs.small[gt] : 0xFFFFFFFFu;
                uint32_t rank = 0;
                for (uint32_t j = 0; j < cnt; ++j) {
                    const uint32_t o = gs.small[j];
                    rank += (o < mine) || (o == mine && j < (uint32_t)gt);
                }
                if ((uint32_t)gt < cnt && rank == krem) gs.r1 = mine;
                if ((uint32_t)gt < cnt && rank == krem + 1) gs.r2 = mine;
            }
            cl_group_bar(barid, G);
            v1 = base + gs.r1;
            if (krem + 1 < cnt) v2 = base + gs.r2;
            else if (gs.vmin != 0xFFFFFFFFu) v2 = base + gs.vmin;
            else { v2 = v1; if (want_next) ok = false; }
            break;
        }
        base += bin << shv;
        // re-base the offsets on the chosen bin: keys outside it drop out
#pragma unroll
        for (int e = 0; e < kClP * JMAX; ++e) {
            const uint32_t o = off[e];
            off[e] = (o <= width && (o >> shv) == bin) ? o - (bin << shv) : 0xFFFFFFFFu;
        }
        width = (1u << shv) - 1u;
        cl_group_bar(barid, G);
        if (round == 3) ok = false;
    }
    cl_group_bar(barid, G);
    return ok;
}

template <int G>
__device__ __forceinline__ bool cl_select_any(const int cap, const ClSegs &sg, uint32_t k, bool want_next, uint32_t base,
                                              uint32_t width, uint32_t *hist, ClSel &gs, int gt, int barid, uint32_t &v1,
                                              uint32_t &v2) {
    if (cap <= 5 * G) return cl_select_regs<G, 5>(sg, k, want_next, base, width, hist, gs, gt, barid, v1, v2);
    return cl_select<G>(sg, k, want_next, base, width, hist, gs, gt, barid, v1, v2);
}

// ---- per-element operations of the sweeps, written out so that each is a fixed handful of
// instructions (compare, predicated add / predicated store) ---------------------------------
// cnt += (x < lo); packed += INC if lo <= x <= hi (NaN is neither).
template <uint32_t INC>
__device__ __forceinline__ void cl_cell_count(const float x, const float lo, const float hi, uint32_t &cnt, uint32_t &packed) {
    asm("{\n\t.reg .pred p, q;\n\tsetp.lt.f32 p, %2, %3;\n\tsetp.le.and.f32 q, %2, %4, !p;\n\t@p add.u32 %0, %0, 1;\n\t@q add.u32 %1, %1, %5;\n\t}"
        : "+r"(cnt), "+r"(packed)
        : "f"(x), "f"(lo), "f"(hi), "n"(INC));
}
// if (lo <= x <= hi) { shared[addr] = x; addr += 4; }
__device__ __forceinline__ void cl_cell_keep(const float x, const float lo, const float hi, uint32_t &addr) {
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ge.f32 p, %1, %2;\n\tsetp.le.and.f32 q, %1, %3, p;\n\t@q st.shared.f32 [%0], %1;\n\t@q add.u32 %0, %0, 4;\n\t}"
                 : "+r"(addr)
                 : "f"(x), "f"(lo), "f"(hi)
                 : "memory");
}
// one step of an inclusive scan over lanes: incl += value of lane (lane - d) where that lane exists
__device__ __forceinline__ void cl_scan_step(uint32_t &incl, const int d) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 r;\n\tshfl.sync.up.b32 r|p, %0, %1, 0, 0xffffffff;\n\t@p add.u32 %0, %0, r;\n\t}"
                 : "+r"(incl)
                 : "r"(d));
}
__device__ __forceinline__ uint32_t cl_atoms_add(const uint32_t addr, const uint32_t v) {
    uint32_t old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}

// Elements that might exceed the threshold (rare): exact tests against the threshold's possible
// range [rlo, rhi]; the bit is set at once or the decision deferred until the MAD is known.
template <int NQ>
__device__ __noinline__ void cl_slow_row(const float *__restrict__ row, const int r, const int q, ClShared &sh, uint32_t *amb,
                                         uint8_t *maskrow) {
    constexpr int M = 4 * NQ;
    const float4 x4 = __ldg(reinterpret_cast<const float4 *>(row + (size_t)r * M) + q);
    const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
    uint32_t eb = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int m = 4 * q + c;
        const float sg = sh.sgn[m];
        const float sdev = __fmaf_rn(xs[c], sg, -sg * sh.med[m]);
        if (sdev > sh.rlo[m]) {
            if (sdev > sh.rhi[m]) {
                eb |= 1u << m;
            } else {
                const uint32_t pos = atomicAdd(&sh.namb, 1u);
                if (pos < (uint32_t)kClAmb) amb[pos] = ((uint32_t)r << 5) | (uint32_t)m;
            }
        }
    }
    if (eb && maskrow) {
        unsigned int *w = reinterpret_cast<unsigned int *>(maskrow + (r & ~3));
        atomicOr(w, eb << (8 * (r & 3)));
    }
}

// One sweep of this CTA's ranks [r0, r1).  MODE 0: count x < lo, keep lo <= x <= hi.
// MODE 1: the same for d = |x - med| against [dlo, dhi], plus the exceedance bits.
// The counts go to the cluster-wide counter of each metric, in its owner's shared memory.
// Kept elements: every batch (kClU ranks x 4 metrics per thread) the lanes of a metric quad
// scan their four 8-bit kept counts (one packed word), the first lane reserves list space for
// all of them with two shared-memory atomics (16-bit counter pairs), and every lane stores
// its kept values at its own offset.  A full list is detected by the owner from the counters;
// stores past the capacity land in the kClSlack words behind each list.
template <int NQ, int MODE>
__device__ __forceinline__ void cl_sweep(const float *__restrict__ row, const int r0, const int r1, const int cap,
                                         ClShared &sh, uint32_t *list, uint32_t *amb, uint8_t *maskrow,
                                         const bool check_finite, uint32_t *status) {
    constexpr int M = 4 * NQ, LPI = kClThreads / NQ, MPC = M / kClP;
    const int tid = threadIdx.x, lane = tid & 31;
    const int q = tid & (NQ - 1), rl = tid / NQ;
    float lo[4], hi[4], sg[4], nsm[4], irlo[4];
    uint32_t cnt[4] = {0, 0, 0, 0};
    bool bad = false;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int m = 4 * q + c;
        if (MODE == 0) {
            lo[c] = sh.lo[m]; hi[c] = sh.hi[m];
            sg[c] = 0.0f; nsm[c] = 0.0f; irlo[c] = 0.0f;
        } else {
            lo[c] = sh.dlo[m]; hi[c] = sh.dhi[m];
            sg[c] = sh.sgn[m];
            nsm[c] = -sg[c] * sh.med[m];
            const float rl_ = sh.rlo[m];
            irlo[c] = rl_ > 0.0f ? 1.0f / rl_ : CUDART_INF_F;
        }
    }
    const uint32_t list_s = (uint32_t)__cvta_generic_to_shared(list) + (uint32_t)(4 * q) * (uint32_t)(cap + kClSlack) * 4u;
    const uint32_t pitch = (uint32_t)(cap + kClSlack) * 4u;   // bytes between the lists of consecutive metrics
    const uint32_t n32_s = (uint32_t)__cvta_generic_to_shared(&sh.n32[2 * q]);
    const uint32_t cap16 = (uint32_t)cap | ((uint32_t)cap << 16);

    auto batch = [&](const int base, const bool guard) {
        float v[kClU][4];
        const float4 *src = reinterpret_cast<const float4 *>(row + (size_t)(base + rl) * M) + q;
#pragma unroll
        for (int j = 0; j < kClU; ++j) {
            float4 x = make_float4(CUDART_NAN_F, CUDART_NAN_F, CUDART_NAN_F, CUDART_NAN_F);
            if (!guard || base + j * LPI + rl < r1) x = __ldg(src + (size_t)j * LPI * NQ);
            v[j][0] = x.x; v[j][1] = x.y; v[j][2] = x.z; v[j][3] = x.w;
        }
        uint32_t packed = 0;
#pragma unroll
        for (int j = 0; j < kClU; ++j) {
            if (MODE == 1) {
                float z[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    // the finite check looks at the value itself: the deviation of two finite values of
                    // opposite sign may overflow
                    const bool nf = nonfinite_bits(__float_as_uint(v[j][c]));
                    const float sdev = __fmaf_rn(v[j][c], sg[c], nsm[c]);
                    const float d = fabsf(sdev);
                    v[j][c] = d;
                    z[c] = sdev * irlo[c];
                    if (guard) bad |= (base + j * LPI + rl < r1) && nf;
                    else bad |= nf;
                }
                // conservative test for "some metric of this rank may exceed": exact tests follow
                if (fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])) > 0.99f && (!guard || base + j * LPI + rl < r1))
                    cl_slow_row<NQ>(row, base + j * LPI + rl, q, sh, amb, maskrow);
            }
            cl_cell_count<1u>(v[j][0], lo[0], hi[0], cnt[0], packed);
            cl_cell_count<1u << 8>(v[j][1], lo[1], hi[1], cnt[1], packed);
            cl_cell_count<1u << 16>(v[j][2], lo[2], hi[2], cnt[2], packed);
            cl_cell_count<1u << 24>(v[j][3], lo[3], hi[3], cnt[3], packed);
        }
        // inclusive scan of the four 8-bit kept counts over the lanes of the same metric quad
        uint32_t incl = packed;
#pragma unroll
        for (int d = NQ; d < 32; d <<= 1) cl_scan_step(incl, d);
        const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 32 - NQ + q);
        uint32_t b01 = 0, b23 = 0;
        if (lane < NQ) {
            b01 = cl_atoms_add(n32_s, __byte_perm(total, 0, 0x4140));
            b23 = cl_atoms_add(n32_s + 4, __byte_perm(total, 0, 0x4342));
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
        for (int j = 0; j < kClU; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) cl_cell_keep(v[j][c], lo[c], hi[c], addr[c]);
    };
    const int span = LPI * kClU;
    int base = r0;
    for (; base + span <= r1; base += span) batch(base, false);
    if (base < r1) batch(base, true);
    // counts below the interval: summed over the lanes of a quad class, then into the owner's counter
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int tot = group_sum<NQ>((int)cnt[c]);
        if (lane < NQ && tot) cl_red_add(cl_map(&sh.cnt[4 * q + c], (4 * q + c) / MPC), (uint32_t)tot);
    }
    if (MODE == 1 && check_finite && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(status, kStatNonFinite);
}

template <int NQ>
__global__ void __cluster_dims__(kClP, 1, 1) __launch_bounds__(kClThreads, 4)
    xrank_cluster_kernel(const XrankArgs a, const MetricParams p, const ClGeom g, uint32_t *reasons) {
    constexpr int M = 4 * NQ, MPC = M / kClP, G = kClThreads / MPC;
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t *list = smem;                         // [M][cap + kClSlack] kept elements of this CTA
    uint32_t *hist = smem + M * (g.cap + kClSlack);   // [MPC][1024] sample / selection histograms
    uint32_t *amb = hist + MPC * kClBins;          // [kClAmb]
    __shared__ ClShared sh;
    __shared__ XrShared xsh;

    const int crank = (int)cg::this_cluster().block_rank();
    const int t = blockIdx.x / kClP, tid = threadIdx.x, lane = tid & 31;
    const int R = a.R;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    uint8_t *maskrow = a.mask_base ? reinterpret_cast<uint8_t *>(a.mask_base) + (size_t)slot * R : nullptr;
    const size_t so = (size_t)t * M;
    const int r0 = min(R, crank * g.slice), r1 = min(R, r0 + g.slice);
    const int grp = tid / G, gt = tid % G, barid = 1 + grp;
    const int m_own = crank * MPC + grp;           // the metric this thread's group selects for
    ClSel &gs = sh.sel[grp];
    uint32_t *h = hist + grp * kClBins;
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2), k2 = (uint32_t)(R / 2);

    // The sample of the owned column (every stride-th rank) and the 32 spread values that fix
    // the bin map are requested first, so that their latency overlaps the set-up below.
    constexpr int SPT = kClSample / G;
    float xs[SPT];
#pragma unroll
    for (int j = 0; j < SPT; ++j) {
        const int i = gt + j * G;
        xs[j] = CUDART_NAN_F;
        if (i < g.s) xs[j] = __ldg(row + (size_t)(i * g.stride + (g.stride >> 1)) * M + m_own);
    }
    float xpre = 0.0f;
    if (gt < 32) xpre = __ldg(row + (size_t)min(R - 1, (int)(((long long)(2 * lane + 1) * R) >> 6)) * M + m_own);

    if (tid < M) { sh.cnt[tid] = 0; sh.sgn[tid] = p.dir[tid] < 0 ? -1.0f : 1.0f; }
    if (tid < 4) sh.n32[tid] = 0u;
    if (tid == 0) { sh.namb = 0; sh.fail = 0; }
    // this CTA's part of the exceedance row starts at zero; bits are OR-ed in
    if (maskrow)
        for (int i = r0 + 4 * tid; i < r1; i += 4 * kClThreads) *reinterpret_cast<uint32_t *>(maskrow + i) = 0u;
    for (int i = gt; i < kClBins; i += G) h[i] = 0;
    cl_sync();   // all four CTAs run and have cleared their state before anyone writes into it

    // ---- 0. sample: histogram of every stride-th rank of the owned column -> intervals -------
    if (gt < 32) {
        const uint32_t key = cl_warp_sort(f2key(xpre), lane);
        const float c50 = key2f(__shfl_sync(0xFFFFFFFFu, key, 16));
        const float c25 = key2f(__shfl_sync(0xFFFFFFFFu, key, 8)), c75 = key2f(__shfl_sync(0xFFFFFFFFu, key, 23));
        if (lane == 0) {
            const float sig = (c75 - c25) / 1.35f;
            const float inv_bw = 64.0f / sig;     // 2048 bins over +-16 sigma
            const float off = (float)(1024.0 - (double)c50 * (double)inv_bw);
            gs.inv_bw = inv_bw;
            gs.off = off;
            gs.sample_ok = (sig > 0.0f) && (inv_bw < kFltMax) && (fabsf(off) < kFltMax);
            const int mid = g.s / 2, q1 = g.s / 4, q3 = (3 * g.s) / 4;
            const int tk[6] = {mid - g.delta, mid + g.delta, q1 - g.delta_q, q1 + g.delta_q, q3 - g.delta_q, q3 + g.delta_q};
#pragma unroll
            for (int i = 0; i < 6; ++i) { gs.tk[i] = (uint32_t)min(max(tk[i], 0), g.s - 1); gs.tb[i] = 0xFFFFFFFFu; }
        }
    }
    cl_group_bar(barid, G);
    const bool sample_ok = gs.sample_ok != 0;
    if (sample_ok) {
        const float inv_bw = gs.inv_bw, off = gs.off;
#pragma unroll
        for (int j = 0; j < SPT; ++j) {
            if (gt + j * G < g.s) {
                int b = __float2int_rd(__fmaf_rn(xs[j], inv_bw, off));
                b = min(max(b, 0), kClSBins - 1);
                atomicAdd(&h[b >> 1], (b & 1) ? 0x10000u : 1u);
            }
        }
    }
    cl_group_bar(barid, G);
    if (sample_ok) {
        // bins of the six sample ranks: scan of the 2048 bin counts, WPT words (2 bins each) per thread
        constexpr int WPT = kClBins / G;
        uint32_t w[WPT], sum = 0;
#pragma unroll
        for (int i = 0; i < WPT; ++i) { w[i] = h[gt * WPT + i]; sum += (w[i] & 0xFFFFu) + (w[i] >> 16); }
        uint32_t incl = sum;
        const int gl = gt & 31, gw = gt >> 5;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (gl >= d) incl += u; }
        if (gl == 31) gs.warp_tot[gw] = incl;
        cl_group_bar(barid, G);
        uint32_t offw = 0;
        for (int ww = 0; ww < gw; ++ww) offw += gs.warp_tot[ww];
        const uint32_t excl = offw + incl - sum;
#pragma unroll
        for (int i6 = 0; i6 < 6; ++i6) {
            const uint32_t k = gs.tk[i6];
            if (k >= excl && k < excl + sum) {
                uint32_t run = excl;
#pragma unroll
                for (int i = 0; i < WPT; ++i) {
                    const uint32_t c0 = w[i] & 0xFFFFu, c1 = w[i] >> 16;
                    if (k >= run && k < run + c0) gs.tb[i6] = (uint32_t)(2 * (gt * WPT + i));
                    run += c0;
                    if (k >= run && k < run + c1) gs.tb[i6] = (uint32_t)(2 * (gt * WPT + i) + 1);
                    run += c1;
                }
            }
        }
    }
    cl_group_bar(barid, G);
    if (gt == 0) {
        bool ok = sample_ok;
#pragma unroll
        for (int i = 0; i < 6; ++i) ok = ok && gs.tb[i] != 0xFFFFFFFFu;
        float lo = 0.0f, hi = 0.0f, dlo = 0.0f, dhi = 0.0f;
        if (ok) {
            // value at the lower edge of bin b under the map x -> x * inv_bw + off
            const double inv = 1.0 / (double)gs.inv_bw, offd = (double)gs.off;
            auto edge = [&](uint32_t b) -> float {
                if (b == 0) return -kFltMax;
                if (b >= (uint32_t)kClSBins) return kFltMax;
                const double e = ((double)b - offd) * inv;
                return (float)fmin(fmax(e, -(double)kFltMax), (double)kFltMax);
            };
            lo = fdown(edge(gs.tb[0]));
            hi = fup(edge(gs.tb[1] + 1));
            if (lo < -kFltMax) lo = -kFltMax;
            if (hi > kFltMax) hi = kFltMax;
            // The MAD is the half-width d at which [med - d, med + d] holds half of the column: the
            // span between the quartiles' outer (inner) neighbours holds more (less) than half with
            // high probability, and for a column roughly symmetric about its median the half-lengths
            // of those spans bracket d.  (A miss is caught by the counts.)
            const float a_lo = edge(gs.tb[2]), a_hi = edge(gs.tb[3] + 1), b_lo = edge(gs.tb[4]), b_hi = edge(gs.tb[5] + 1);
            const float d0 = 0.5f * (b_lo - a_hi), d1 = 0.5f * (b_hi - a_lo);
            dlo = d0 > 0.0f ? fdown(d0) : 0.0f;
            dhi = (d1 >= 0.0f && d1 < kFltMax) ? fup(d1) : kFltMax;
            if (dhi > kFltMax) dhi = kFltMax;
        }
#pragma unroll
        for (int c = 0; c < kClP; ++c) {
            cl_stf(cl_map(&sh.lo[m_own], c), lo); cl_stf(cl_map(&sh.hi[m_own], c), hi);
            cl_stf(cl_map(&sh.dlo[m_own], c), dlo); cl_stf(cl_map(&sh.dhi[m_own], c), dhi);
            if (!ok) cl_red_max(cl_map(&sh.fail, c), 2);
        }
        if (!ok && reasons) atomicAdd(reasons + kWhySelect, 1u);
    }
    cl_sync();   // intervals known everywhere, counters zeroed

    int verdict = sh.fail;
    // ---- 1./2. median: sweep, select ----------------------------------------------------------
    for (int attempt = 0; verdict == 0; ++attempt) {
        cl_sweep<NQ, 0>(row, r0, r1, g.cap, sh, list, amb, maskrow, false, a.status);
        cl_sync();
        {
            const int m = m_own;
            ClSegs sg;
            uint32_t n = 0;
            bool over = false;
#pragma unroll
            for (int c = 0; c < kClP; ++c) {
                sg.p[c] = cl_map(list + m * (g.cap + kClSlack), c);
                sg.n[c] = (cl_ld(cl_map(&sh.n32[m >> 1], c)) >> (16 * (m & 1))) & 0xFFFFu;
                over |= sg.n[c] > (uint32_t)g.cap;
                n += sg.n[c];
            }
            const uint32_t clt = sh.cnt[m];
            int why = -1, shift = 0;
            if (over) why = kWhyCtaList;
            else if (clt > k1) { why = kWhyMedianMiss; shift = -1; }
            else if (k2 >= clt + n) { why = kWhyMedianMiss; shift = 1; }
            uint32_t v1 = 0, v2 = 0;
            const float flo = sh.lo[m], fhi = sh.hi[m];
            if (why < 0) {
                const uint32_t base = f2key(flo == 0.0f ? -0.0f : flo);
                const uint32_t width = f2key(fhi == 0.0f ? 0.0f : fhi) - base;
                if (!cl_select_any<G>(g.cap, sg, k1 - clt, even, base, width, h, gs, gt, barid, v1, v2)) why = kWhySelect;
            }
            cl_group_bar(barid, G);   // every thread of the group has read the count before it is cleared
            if (gt == 0) {
                sh.cnt[m] = 0;
                if (why < 0) {
                    const float med = median_from_keys(v1, v2, even);
                    a.med[so + m] = med;
                    if (a.med_user) a.med_user[so + m] = med;
                    const float rel = __fmul_rn(p.floor_rel[m], fabsf(med));
                    const float rlo = __fmul_rn(p.thrp[m], fmaxf(fmaxf(sh.dlo[m], rel), p.floor_abs[m]));
                    const float rhi = __fmul_rn(p.thrp[m], fmaxf(fmaxf(sh.dhi[m], rel), p.floor_abs[m]));
#pragma unroll
                    for (int c = 0; c < kClP; ++c) {
                        cl_stf(cl_map(&sh.med[m], c), med); cl_stf(cl_map(&sh.rlo[m], c), rlo); cl_stf(cl_map(&sh.rhi[m], c), rhi);
                    }
                } else {
                    if (reasons) atomicAdd(reasons + why, 1u);
                    const int v = (shift != 0 && attempt == 0) ? 1 : 2;
                    // the counts say on which side of its interval the middle lies: move the interval
                    // by its own width (the kept lists cannot hold a wider one)
                    const float w = fhi - flo;
                    float nlo = flo, nhi = fhi;
                    if (shift < 0) { nhi = flo; nlo = fmaxf(flo - w, -kFltMax); }
                    if (shift > 0) { nlo = fhi; nhi = fminf(fhi + w, kFltMax); }
#pragma unroll
                    for (int c = 0; c < kClP; ++c) {
                        cl_stf(cl_map(&sh.lo[m], c), nlo); cl_stf(cl_map(&sh.hi[m], c), nhi);
                        cl_red_max(cl_map(&sh.fail, c), v);
                    }
                }
            }
        }
        cl_sync();
        verdict = sh.fail;
        __syncthreads();   // everyone has read the verdict and the kept counts are no longer needed
        if (tid < 4) sh.n32[tid] = 0u;
        if (verdict != 1) break;
        if (tid == 0) sh.fail = 0;
        cl_sync();    // cleared everywhere before the next attempt's verdicts can arrive
        verdict = 0;
    }
    // ---- 3./4. MAD + exceedance: sweep, select ------------------------------------------------
    if (verdict == 0) {
        __syncthreads();
        for (int attempt = 0;; ++attempt) {
            cl_sweep<NQ, 1>(row, r0, r1, g.cap, sh, list, amb, maskrow, a.check_finite != 0, a.status);
            cl_sync();
            {
                const int m = m_own;
                ClSegs sg;
                uint32_t n = 0;
                bool over = false, amb_over = false;
#pragma unroll
                for (int c = 0; c < kClP; ++c) {
                    sg.p[c] = cl_map(list + m * (g.cap + kClSlack), c);
                    sg.n[c] = (cl_ld(cl_map(&sh.n32[m >> 1], c)) >> (16 * (m & 1))) & 0xFFFFu;
                    over |= sg.n[c] > (uint32_t)g.cap;
                    amb_over |= cl_ld(cl_map(&sh.namb, c)) > (uint32_t)kClAmb;
                    n += sg.n[c];
                }
                const uint32_t clt = sh.cnt[m];
                int why = -1, shift = 0;
                if (amb_over) why = kWhyAmbList;
                else if (over) why = kWhyCtaList;
                else if (clt > k1) { why = kWhyMadMiss; shift = -1; }
                else if (k2 >= clt + n) { why = kWhyMadMiss; shift = 1; }
                uint32_t v1 = 0, v2 = 0;
                const float flo = sh.dlo[m], fhi = sh.dhi[m];
                if (why < 0) {
                    const uint32_t base = f2key(flo);
                    const uint32_t width = f2key(fhi) - base;
                    if (!cl_select_any<G>(g.cap, sg, k1 - clt, even, base, width, h, gs, gt, barid, v1, v2)) why = kWhySelect;
                }
                cl_group_bar(barid, G);
                if (gt == 0) {
                    sh.cnt[m] = 0;
                    if (why < 0) {
                        const float mad = median_from_keys(v1, v2, even);
                        a.mad[so + m] = mad;
                        if (a.mad_user) a.mad_user[so + m] = mad;
                        const float rhs = __fmul_rn(p.thrp[m], scale_of(mad, sh.med[m], p.floor_rel[m], p.floor_abs[m]));
#pragma unroll
                        for (int c = 0; c < kClP; ++c) cl_stf(cl_map(&sh.rhs[m], c), rhs);
                    } else {
                        if (reasons) atomicAdd(reasons + why, 1u);
                        const int v = (shift != 0 && attempt == 0) ? 1 : 2;
                        const float w = fhi - flo;
                        float nlo = flo, nhi = fhi;
                        if (shift < 0) { nhi = flo; nlo = fmaxf(0.0f, flo - w); }
                        if (shift > 0) { nlo = fhi; nhi = fminf(fhi + w, kFltMax); }
                        const float rel = __fmul_rn(p.floor_rel[m], fabsf(sh.med[m]));
                        const float rlo = __fmul_rn(p.thrp[m], fmaxf(fmaxf(nlo, rel), p.floor_abs[m]));
                        const float rhi = __fmul_rn(p.thrp[m], fmaxf(fmaxf(nhi, rel), p.floor_abs[m]));
#pragma unroll
                        for (int c = 0; c < kClP; ++c) {
                            cl_stf(cl_map(&sh.dlo[m], c), nlo); cl_stf(cl_map(&sh.dhi[m], c), nhi);
                            cl_stf(cl_map(&sh.rlo[m], c), rlo); cl_stf(cl_map(&sh.rhi[m], c), rhi);
                            cl_red_max(cl_map(&sh.fail, c), v);
                        }
                    }
                }
            }
            cl_sync();
            verdict = sh.fail;
            __syncthreads();
            if (verdict != 1) break;
            // Sweep again with the moved intervals.  Exceedance bits already set stay valid only if
            // they are set again, so the row part and the deferred list start over.
            if (tid < 4) sh.n32[tid] = 0u;
            if (tid == 0) { sh.fail = 0; sh.namb = 0; }
            if (maskrow)
                for (int i = r0 + 4 * tid; i < r1; i += 4 * kClThreads) *reinterpret_cast<uint32_t *>(maskrow + i) = 0u;
            cl_sync();
        }
    }
    if (verdict == 0) {
        // ---- 5. deferred exceedance decisions of this CTA's ranks ------------------------------
        if (maskrow) {
            const uint32_t na = sh.namb;
            for (uint32_t i = tid; i < na; i += kClThreads) {
                const uint32_t e = amb[i];
                const uint32_t r = e >> 5, m = e & 31u;
                if (exceeds(row[(size_t)r * M + m], sh.med[m], p.dir[m], sh.rhs[m])) {
                    unsigned int *w = reinterpret_cast<unsigned int *>(maskrow + (r & ~3u));
                    atomicOr(w, (1u << m) << (8 * (r & 3u)));
                }
            }
        }
        return;
    }
    // ---- fallback: the first CTA recomputes the whole step with the direct radix select --------
    if (crank != 0) return;
    __syncthreads();
    xrank_direct_step(a, p, t, smem, xsh);
    if (tid == 0 && a.fallbacks) atomicAdd(a.fallbacks, 1u);
}

// Kept fraction of a column: the median interval spans 2 delta of s sample ranks, the MAD
// interval 4 delta_q (one band around each quartile), plus the bins the interval ends are
// rounded to.
ClGeom cluster_geometry(int R, int M) {
    ClGeom g{};
    g.slice = ((R + kClP - 1) / kClP + 15) / 16 * 16;
    g.stride = (R + kClSample - 1) / kClSample;
    if (g.stride < 1) g.stride = 1;
    g.s = (R - (g.stride >> 1) + g.stride - 1) / g.stride;
    const double sq = sqrt((double)g.s);
    g.delta = (int)ceil(5.5 * 0.5 * sq);
    g.delta_q = (int)ceil(0.5 * 4.0 * 0.612 * sq);
    const double f_med = 2.0 * g.delta / g.s, f_mad = 4.0 * g.delta_q / g.s;
    const double f = (f_med > f_mad ? f_med : f_mad) + 0.02;
    g.cap = (int)ceil(g.slice * f * 1.25) + 64;
    g.cap = (g.cap + 31) / 32 * 32;
    if (g.cap < 256) g.cap = 256;
    (void)M;
    return g;
}

size_t cluster_smem(const ClGeom &g, int M) {
    return (size_t)(M * (g.cap + kClSlack) + (M / kClP) * kClBins + kClAmb) * sizeof(uint32_t);
}

}  // namespace

bool xrank_cluster_supported(int R, int M) {
    if (M != 4 && M != 8) return false;
    if (R < 4096 || (R & 3) != 0 || R > 4 * 32768) return false;
    const ClGeom g = cluster_geometry(R, M);
    return cluster_smem(g, M) <= 96 * 1024;
}

cudaError_t launch_xrank_cluster(const XrankArgs &a, const MetricParams &p, int S, uint32_t *reasons, cudaStream_t st,
                                 std::vector<std::pair<cudaEvent_t, cudaEvent_t>> *prof) {
    if (S <= 0) return cudaSuccess;
    const ClGeom g = cluster_geometry(a.R, a.M);
    const size_t smem = cluster_smem(g, a.M);
    cudaError_t e;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (prof) {
        if (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess) return cudaGetLastError();
        cudaEventRecord(ev0, st);
    }
    if (a.M == 8) {
        e = cudaFuncSetAttribute(xrank_cluster_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        xrank_cluster_kernel<2><<<S * kClP, kClThreads, smem, st>>>(a, p, g, reasons);
    } else {
        e = cudaFuncSetAttribute(xrank_cluster_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        xrank_cluster_kernel<1><<<S * kClP, kClThreads, smem, st>>>(a, p, g, reasons);
    }
    e = cudaGetLastError();
    if (prof) {
        cudaEventRecord(ev1, st);
        prof->emplace_back(ev0, ev1);
    }
    return e;
}

}  // namespace guard
