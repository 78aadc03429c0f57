// Windowed per-series median: for every (rank, metric) series the exact median of its
// last n ring steps.  A CTA stages a [n steps] x [TC series] tile of the ring in shared
// memory with bulk asynchronous copies (one per ring row, completion on an mbarrier),
// then every thread selects inside its own column.
#include <math_constants.h>

#include <mutex>

#include "colselect.cuh"
#include "kernels.h"
#include "thselect.cuh"
#include "warpselect.cuh"
#include "xrank_common.cuh"

namespace guard {

namespace {

constexpr size_t kMaxStagedTile = 200 * 1024;   // largest staged tile (dynamic shared memory of the staged path)

// Staged path.  blockDim.x == TC; dynamic shared memory = n * TC * 4 bytes.
template <int TC>
__global__ void __launch_bounds__(TC) window_select_kernel(const WindowArgs a, const int use_bulk) {
    extern __shared__ __align__(128) uint32_t tile[];
    __shared__ __align__(8) uint64_t bar;
    const int tid = threadIdx.x;
    const int col0 = blockIdx.x * TC;
    const int ncols = min(TC, a.series - col0);
    const int n = a.n;
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;

    if (use_bulk) {
        if (tid == 0) {
            mbar_init(&bar, 1);
            mbar_arrive_expect_tx(&bar, (uint32_t)n * (uint32_t)ncols * 4u);
        }
        __syncthreads();
        for (int j = tid; j < n; j += TC) {
            int slot = first + j;
            if (slot >= a.capacity) slot -= a.capacity;
            bulk_g2s(tile + (size_t)j * TC, a.ring + (size_t)slot * a.row_stride + col0, (uint32_t)ncols * 4u, &bar);
        }
        if (!mbar_wait_bounded(&bar, 0, kWaitLimitCycles)) {
            atomicOr(a.status, kStatTimeout);
            mbar_wait_bounded(&bar, 0, kWaitLimitCycles);  // let copies in flight land before leaving
            return;
        }
    } else {
        for (int j = 0; j < n; ++j) {
            int slot = first + j;
            if (slot >= a.capacity) slot -= a.capacity;
            if (tid < ncols)
                tile[(size_t)j * TC + tid] = __float_as_uint(a.ring[(size_t)slot * a.row_stride + col0 + tid]);
        }
        // each thread only reads back what it wrote itself: no barrier needed
    }
    if (tid >= ncols) return;
    uint32_t *col = tile + tid;
    for (int j = 0; j < n; j += kSelBatch) {   // raw bits -> order-preserving keys, loads batched
        uint32_t v[kSelBatch];
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) v[u] = (j + u < n) ? col[(size_t)(j + u) * TC] : 0u;
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u)
            if (j + u < n) col[(size_t)(j + u) * TC] = key_of_bits(v[u]);
    }
    const float med = col_median(col, TC, n);
    a.wmed[col0 + tid] = med;
    if (a.wmed_user) a.wmed_user[col0 + tid] = med;
}

// ---------------------------------------------------------------------------------------
// Warp-per-series path for windows of up to 256 steps: the window of one series lives in
// the registers of one warp (VPL keys per lane), so no shared-memory column limits the
// number of resident warps.  A CTA of 32 warps handles a tile of 32 adjacent series; tiles
// are staged into a double buffer with one bulk asynchronous copy (TMA) per ring row onto
// an mbarrier per buffer (plain cp.async when rows are not 16-byte aligned).  Rows are
// pitched 36 words apart: 16-byte aligned for the bulk copy, and a column read then costs
// four shared-memory wavefronts instead of thirty-two.
//
// Selection: every lane sorts its own keys (odd-even merge network).  The median of the
// lanes' middle keys (a 32-key bitonic sort over shuffles) is a pivot within a few ranks of
// the wanted one; every lane counts its keys below / not above the pivot and one
// __reduce_add_sync gives the pivot's global rank.  From there the warp walks rank by rank
// (each lane offers its next key, __reduce_min/max_sync picks the winner) until it passes
// the wanted rank; if the pivot turns out to be far off, further pivot rounds (middle key of
// the longest still-active run) narrow the distance first.  Every round removes at least its
// pivot from the active set, so the loop is bounded by the window length.
// ---------------------------------------------------------------------------------------
constexpr int kWarpTileCols = 32;
constexpr int kWarpPitch = 36;

__device__ __forceinline__ void cp_async4(void *dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

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

template <int VPL>
__global__ void __launch_bounds__(1024, 2) window_warp_kernel(const WindowArgs a, const int ntiles, const int use_bulk) {
    extern __shared__ __align__(128) uint32_t wbuf[];   // 2 x [n][kWarpPitch]
    __shared__ __align__(8) uint64_t bar[2];
    const int tid = threadIdx.x, lane = lane_id(), w = warp_id();
    const int n = a.n;
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;
    const int bufwords = n * kWarpPitch;

    auto stage = [&](int tile, int b) {
        uint32_t *buf = wbuf + b * bufwords;
        const int col0 = tile * kWarpTileCols;
        const int ncols = min(kWarpTileCols, a.series - col0);
        if (use_bulk) {
            if (tid == 0) mbar_arrive_expect_tx(&bar[b], (uint32_t)n * (uint32_t)ncols * 4u);
            __syncthreads();   // the expectation is registered before any copy can complete
            // lane l of warp w issues rows w + 32 l, w + 32 l + 1024, ...: a warp's bulk copies are
            // issued one lane after the other, so they are spread over all warps
            for (int row = w + 32 * lane; row < n; row += 1024) {
                int slot = first + row;
                if (slot >= a.capacity) slot -= a.capacity;
                bulk_g2s(buf + row * kWarpPitch, a.ring + (size_t)slot * a.row_stride + col0, (uint32_t)ncols * 4u, &bar[b]);
            }
        } else {
            for (int e = tid; e < n * kWarpTileCols; e += 1024) {
                const int row = e >> 5, c = e & 31;
                int slot = first + row;
                if (slot >= a.capacity) slot -= a.capacity;
                if (c < ncols) cp_async4(buf + row * kWarpPitch + c, a.ring + (size_t)slot * a.row_stride + col0 + c);
            }
            cp_async_commit();
        }
    };

    if (use_bulk && tid == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
    }
    __syncthreads();
    int cur = 0, it = 0;
    if ((int)blockIdx.x < ntiles) stage(blockIdx.x, 0);
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
        const int next = tile + gridDim.x;
        if (next < ntiles) stage(next, cur ^ 1);
        if (use_bulk) {
            // only this first wait takes the caller's (test) limit: the waits below, which let the copies
            // in flight land before the CTA leaves, always get the full one.  The CTA decides as one:
            // if the wait ran out for any thread, all of them leave.
            const bool arrived = mbar_wait_bounded(&bar[cur], (uint32_t)((it >> 1) & 1),
                                                   a.first_wait_cycles > 0 ? a.first_wait_cycles : kWaitLimitCycles);
            if (__syncthreads_or(!arrived)) {
                if (!arrived) atomicOr(a.status, kStatTimeout);
                mbar_wait_bounded(&bar[cur], (uint32_t)((it >> 1) & 1), kWaitLimitCycles);   // let copies in flight land
                if (next < ntiles) mbar_wait_bounded(&bar[cur ^ 1], (uint32_t)(((it + 1) >> 1) & 1), kWaitLimitCycles);
                return;
            }
        } else {
            if (next < ntiles) cp_async_wait<1>(); else cp_async_wait<0>();
            __syncthreads();
        }
        const uint32_t *buf = wbuf + cur * bufwords;
        const int series = tile * kWarpTileCols + w;
        if (series < a.series) {
            uint32_t kv[VPL];
            int nreal = 0;
#pragma unroll
            for (int i = 0; i < VPL; ++i) {
                const int row = lane + 32 * i;
                const bool real = row < n;
                kv[i] = real ? key_of_bits(buf[row * kWarpPitch + w]) : 0xFFFFFFFFu;
                nreal += real;
            }
            lane_sort<VPL>(kv);
            float med = 0.0f;
            const uint32_t hint = (a.use_hint && a.wmed_prev) ? f2key(a.wmed_prev[series]) : 0u;   // last evaluation's median
            const bool ok = warp_median<VPL>(kv, nreal, n, hint, med);
            const float h0 = warp_spread_guess<VPL>(kv, n, med);
            if (lane == 0) {
                if (!ok) atomicOr(a.status, kStatInternal);
                a.wmed[series] = med;
                if (a.wmed_user) a.wmed_user[series] = med;
                if (a.spread) a.spread[series] = h0;
                if (a.centre) a.centre[series] = med;
            }
        }
        __syncthreads();   // every warp is done with this buffer before it is refilled
        cur ^= 1;
    }
}

// Function attributes are set once per device and kernel (the calls go to the driver: two of them
// per evaluation showed in the per-step latency of the streaming configuration).
struct AttrOnce {
    std::mutex mu;
    bool done[64] = {};
    int sms[64] = {};
    template <typename F>
    cudaError_t operator()(int &dev_out, F &&set) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        dev_out = dev & 63;
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev_out]) {
            e = set();
            if (e != cudaSuccess) return e;
            if (cudaDeviceGetAttribute(&sms[dev_out], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms[dev_out] = 148;
            done[dev_out] = true;
        }
        return cudaSuccess;
    }
};

template <int VPL>
cudaError_t launch_warp_path(const WindowArgs &a, int use_bulk, cudaStream_t st) {
    const size_t smem = 2 * (size_t)a.n * kWarpPitch * 4;
    static AttrOnce once;
    int dev = 0;
    cudaError_t e = once(dev, [] {
        return cudaFuncSetAttribute(window_warp_kernel<VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 32 * VPL * kWarpPitch * 4);
    });
    if (e != cudaSuccess) return e;
    const int sms = once.sms[dev];
    const int ntiles = (a.series + kWarpTileCols - 1) / kWarpTileCols;
    const int grid = ntiles < 2 * sms ? ntiles : 2 * sms;
    window_warp_kernel<VPL><<<grid, 1024, smem, st>>>(a, ntiles, use_bulk);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Thread path: from the second evaluation on, a series' smoothed median and a tuned half-width
// h give an interval [centre - h, centre + h] that almost always holds the new middle
// elements, so that counting the values below the interval and selecting among the few dozen
// inside it replaces sorting the window.  One thread per series reads its window
// straight from the ring (a warp reads 32 adjacent series of a row: one fully used 128-byte
// line per load, eight rows in flight per thread), counts the values below the interval and
// keeps those inside it, as raw bits, in its own shared-memory column.  No thread ever waits
// for another one: there is no barrier in the kernel, CTAs are four warps, and with 60 kept
// slots per thread seven CTAs share an SM.  The interval is centred on a smoothed median (a
// single window's median carries its own sampling noise, which would add to the next one's).
//
// Selection among the kept keys runs the same instruction stream in every lane: the column
// is turned into order-preserving keys once (128-bit shared-memory accesses; a column is 60
// words, 4 x an odd number, so the lanes' quads fall on different banks), then counting
// passes (keys below a pivot interpolated between the ends of a shrinking key bracket, every
// third pass a bisection) run until t - 1, t or t + 1 keys lie below the pivot: the two
// largest keys below it and the two smallest not below it then include ranks t - 1 and t.
// If the bracket shrinks to one key, that key holds both ranks (ties).
// A series whose interval missed, overflowed or did not converge is finished by its whole
// warp: the lanes fetch the window (L2 hits), sort in registers and run the warp selection.
// ---------------------------------------------------------------------------------------
constexpr int kThCols = 128;     // series per CTA = threads per CTA
constexpr int kThSlots = 60;     // kept keys per series
constexpr int kThTarget = 42;    // number of keys the interval is tuned to catch (windows that share few steps)
constexpr int kThRows = 8;       // rows in flight per thread
constexpr int kThMaxPasses = 12;
constexpr float kThSmooth = 0.3f;   // weight of the newest median in the interval's centre

template <int VPL>
__global__ void __launch_bounds__(kThCols, 9) window_thread_kernel(const WindowArgs a) {
    extern __shared__ __align__(16) uint32_t tkept[];   // [kThCols][kThSlots]
    const int tid = threadIdx.x, lane = lane_id();
    const int n = a.n;
    const int c = blockIdx.x * kThCols + tid;
    const bool active = c < a.series;
    const int cc = active ? c : a.series - 1;           // idle lanes of the last CTA read a valid column
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;
    const int n1 = min(n, a.capacity - first);          // rows before the ring wraps

    const float hint = a.centre[cc], h = a.spread[cc];
    const bool usable = active && (h > 0.0f) && (h < 3.0e38f) && (fabsf(hint) < 3.0e38f);
    // Float compares agree with the key order as long as an end that is zero admits both zeros
    // (-0 as lower end, +0 as upper end).  An unusable interval keeps and counts nothing.
    float flo = hint - h, fhi = hint + h;
    if (flo == 0.0f) flo = -0.0f;
    if (fhi == 0.0f) fhi = 0.0f;
    if (!usable) { flo = CUDART_INF_F; fhi = -CUDART_INF_F; }
    const uint32_t klo = usable ? f2key(flo) : 0xFFFFFFFFu, khi = usable ? f2key(fhi) : 0u;

    const uint32_t kbase = smem_u32(tkept + tid * kThSlots), klim = kbase + (uint32_t)(kThSlots * 4);
    uint32_t kaddr = kbase, clt = 0;
    auto stream = [&](const float *__restrict__ p, const int rows) {
        int r = 0;
        for (; r + kThRows <= rows; r += kThRows) {
            float x[kThRows];
#pragma unroll
            for (int u = 0; u < kThRows; ++u) x[u] = __ldg(p + (size_t)(r + u) * a.row_stride);
#pragma unroll
            for (int u = 0; u < kThRows; ++u) th_cell(x[u], flo, fhi, klim, clt, kaddr);
        }
        for (; r < rows; ++r) th_cell(__ldg(p + (size_t)r * a.row_stride), flo, fhi, klim, clt, kaddr);
    };
    stream(a.ring + (size_t)first * a.row_stride + cc, n1);
    stream(a.ring + cc, n - n1);

    const bool even = !(n & 1);
    const int k1 = (n - 1) >> 1, k2 = n >> 1;
    const int nk = (int)((kaddr - kbase) >> 2);
    bool ok = usable && (int)clt <= k1 && k2 < (int)clt + nk && nk <= kThSlots;
    const int t = k2 - (int)clt;     // rank of the upper middle among the kept keys (t >= 1 when n is even)
    float med = 0.0f;
    // ---- selection among the kept keys: the same instruction stream in every lane ---------------
    uint32_t vb = 0, vu = 0;
    th_select_pair<kThSlots, kThMaxPasses>(kbase, nk, ok, t, klo, khi, vb, vu);
    if (ok) med = median_from_keys(even ? vb : vu, vu, even);
    if (active && ok) {
        a.wmed[c] = med;
        if (a.wmed_user) a.wmed_user[c] = med;
        // re-tune the half-width so that the interval catches about kThTarget keys next time
        // (half of the way: one window's count is a noisy estimate of the density)
        const float f = fminf(2.0f, fmaxf(0.5f, (float)(a.target > 0 ? a.target : kThTarget) / (float)max(nk, 1)));
        a.spread[c] = h * (0.5f + 0.5f * f);
        a.centre[c] = hint + (a.smooth > 0.0f ? a.smooth : kThSmooth) * (med - hint);
    }
    // ---- series the interval did not serve go on the launch's list (window_finish_kernel follows) ------
    // why (diagnostic): 0 no usable interval, 1 more keys than slots, 2 median below the interval,
    // 3 above it, 4 selection did not converge
    const int why = !usable ? 0 : (nk > kThSlots ? 1 : ((int)clt > k1 ? 2 : (k2 >= (int)clt + nk ? 3 : 4)));
    const unsigned todo = __ballot_sync(0xFFFFFFFFu, active && !ok);
    if (todo) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(a.fb_list_count, (uint32_t)__popc(todo));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if ((todo >> lane) & 1u) a.fb_list[base + __popc(todo & ((1u << lane) - 1u))] = ((uint32_t)why << 28) | (uint32_t)c;
    }
}

// The series the thread path's interval did not serve (a few per thousand), one warp per listed series: the lanes
// fetch the window, sort their own keys and run the warp selection; the series' interval state starts afresh.
// A kernel of its own, so that these series spread over the GPU instead of queueing behind one another at the end
// of the warp that found them.
constexpr int kFinThreads = 128;
constexpr int kFinCtas = 148 * 4;

template <int VPL>
__global__ void __launch_bounds__(kFinThreads) window_finish_kernel(const WindowArgs a) {
    __shared__ int is_last;
    const int lane = lane_id();
    const int n = a.n;
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;
    const uint32_t count = min(__ldcg(a.fb_list_count), (uint32_t)a.series);
    const uint32_t nwarps = gridDim.x * (kFinThreads / 32);
    for (uint32_t i = blockIdx.x * (kFinThreads / 32) + warp_id(); i < count; i += nwarps) {
        const uint32_t item = __ldcg(a.fb_list + i);
        const int series = (int)(item & 0x0FFFFFFFu), why_src = (int)(item >> 28);
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
    // the CTA that finishes last clears the list for the next launch
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(a.fb_list_count + 1, 1u) == gridDim.x - 1u) ? 1 : 0;
    __syncthreads();
    if (is_last && threadIdx.x == 0) {
        a.fb_list_count[0] = 0u;
        a.fb_list_count[1] = 0u;
    }
}

template <int VPL>
cudaError_t launch_thread_path(const WindowArgs &a, cudaStream_t st) {
    const size_t smem = (size_t)kThSlots * kThCols * 4;
    static AttrOnce once;
    int dev = 0;
    cudaError_t e = once(dev, [] {
        cudaError_t e2 = cudaFuncSetAttribute(window_thread_kernel<VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, kThSlots * kThCols * 4);
        if (e2 == cudaSuccess)
            e2 = cudaFuncSetAttribute(window_thread_kernel<VPL>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        return e2;
    });
    if (e != cudaSuccess) return e;
    window_thread_kernel<VPL><<<(a.series + kThCols - 1) / kThCols, kThCols, smem, st>>>(a);
    const int fgrid = min(kFinCtas, (a.series + kFinThreads / 32 - 1) / (kFinThreads / 32));
    window_finish_kernel<VPL><<<fgrid, kFinThreads, 0, st>>>(a);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Sliding-window path: evaluations that follow one another by a few steps (streaming: one step)
// share all but a few steps of their windows, so a series' median moves by a rank or two.  Each
// series keeps, across evaluations, an interval [lo, hi] around its median, the number of window
// values below lo, and the handful of values inside the interval (global memory, each series' sorted
// list contiguous).  An evaluation reads only the steps that entered and left the window, one thread
// per series: a value below lo moves the count; a value inside the interval is inserted into /
// removed from the series' list by the whole warp (lane j holds list slots j and j + 32: the position
// comes from a ballot, the shift from one shuffle), series after series; the median is then
// position (middle - count) of the list.
// A series whose median has left its interval, whose list is full, or that has no state yet is
// rebuilt by its whole warp: the lanes fetch the window, sort it (bitonic network over registers
// and shuffles) and take the median, the interval ends kIncHalf ranks beyond the middle ranks, and
// the values inside.  Exact either way: the interval only decides which values are listed.
// ---------------------------------------------------------------------------------------
constexpr int kIncThreads = 128;

// NEW: the most steps that entered / left (1 for an evaluation after every step, else kIncMaxNew).
template <int NEW>
__global__ void __launch_bounds__(kIncThreads, 8) window_inc_kernel(const WindowArgs a, const IncArgs s) {
    static_assert(kIncSlots > 32 && kIncSlots <= 64, "a lane holds list slots lane and lane + 32");
    __shared__ float sl[kIncThreads / 32][32][kIncSlots];   // per warp: the lists of the series it updates, staged asynchronously
    const int lane = lane_id(), wid = warp_id();
    const int n = a.n;
    const int c = blockIdx.x * kIncThreads + threadIdx.x;
    const bool active = c < a.series;
    const int cc = active ? c : a.series - 1;
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;   // slot of the window's oldest step
    const bool even = !(n & 1);
    const int k1 = (n - 1) >> 1, k2 = n >> 1;

    const uint32_t w = s.cnt[cc];
    bool ok = active && (w >> 31) && !s.rebuild_all;
    int cb = (int)(w & 0xFFFFu), nin = (int)((w >> 16) & 0xFFu);
    const float lo = s.lo[cc], hi = s.hi[cc];
    // The steps that left the window (the ones right before its oldest step) and the steps that entered it (the
    // newest ones), all fetched up front.  A value below lo moves the count; a value inside the interval
    // changes the series' sorted list, which the whole warp then updates (below).
    float xl[NEW], xe[NEW];
    uint32_t in_l = 0, in_e = 0;   // which of them lie inside the interval
#pragma unroll
    for (int i = 0; i < NEW; ++i) {
        xl[i] = 0.0f;
        xe[i] = 0.0f;
        if (i < s.leaving) {
            int slot = first - s.leaving + i;
            if (slot < 0) slot += a.capacity;
            xl[i] = __ldg(a.ring + (size_t)slot * a.row_stride + cc);
        }
        if (i < s.entering) {
            int slot = a.last_slot - (s.entering - 1 - i);
            if (slot < 0) slot += a.capacity;
            xe[i] = __ldg(a.ring + (size_t)slot * a.row_stride + cc);
        }
    }
#pragma unroll
    for (int i = 0; i < NEW; ++i) {
        if (i < s.leaving) {
            if (xl[i] < lo) --cb;
            else if (xl[i] <= hi) in_l |= 1u << i;
        }
        if (i < s.entering) {
            if (xe[i] < lo) ++cb;
            else if (xe[i] <= hi) in_e |= 1u << i;
        }
    }
    // ---- list updates, one series at a time by the whole warp: lane j holds list slots j and j + 32 ----
    float f1 = 0.0f, f2 = 0.0f;
    bool have = false;             // f1 / f2 hold the list values at the middle ranks
    unsigned upd = __ballot_sync(0xFFFFFFFFu, ok && (in_l | in_e) != 0u);
    {   // all lists this warp needs are fetched at once (asynchronous copies into shared memory: one round trip)
        unsigned m = upd;
        int k = 0;
        while (m) {
            const int src = __ffs(m) - 1;
            m &= m - 1;
            const int cs = __shfl_sync(0xFFFFFFFFu, c, src);
            const int ns = __shfl_sync(0xFFFFFFFFu, nin, src);
            const float *g = s.val + (size_t)cs * kIncSlots;   // a series' list is contiguous
            if (lane < ns) cp_async4(&sl[wid][k][lane], g + lane);
            if (lane + 32 < ns) cp_async4(&sl[wid][k][lane + 32], g + lane + 32);
            ++k;
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
    }
    int kk = 0;
    while (upd) {
        const int src = __ffs(upd) - 1;
        upd &= upd - 1;
        const int cs = __shfl_sync(0xFFFFFFFFu, c, src);
        int ns = __shfl_sync(0xFFFFFFFFu, nin, src);
        const uint32_t ml = __shfl_sync(0xFFFFFFFFu, in_l, src), me = __shfl_sync(0xFFFFFFFFu, in_e, src);
        const size_t lbase = (size_t)cs * kIncSlots;
        const float v0s = sl[wid][kk][lane], v1s = sl[wid][kk][(lane + 32) % kIncSlots];
        float v0 = lane < ns ? v0s : 0.0f, v1 = lane + 32 < ns ? v1s : 0.0f;
        ++kk;
        bool good = true;
        int dirty_from = kIncSlots;
#pragma unroll
        for (int i = 0; i < NEW; ++i) {
            const float x = __shfl_sync(0xFFFFFFFFu, xl[i], src);
            if (!((ml >> i) & 1u) || !good) continue;    // uniform: ml and good are the same in every lane
            const uint32_t m0 = __ballot_sync(0xFFFFFFFFu, lane < ns && __float_as_uint(v0) == __float_as_uint(x));
            const uint32_t m1 = __ballot_sync(0xFFFFFFFFu, lane + 32 < ns && __float_as_uint(v1) == __float_as_uint(x));
            if ((m0 | m1) == 0u) { good = false; continue; }   // the books do not balance: rebuild
            const int pos = m0 ? __ffs(m0) - 1 : 32 + __ffs(m1) - 1;
            // positions above pos move down by one
            const float d0 = __shfl_down_sync(0xFFFFFFFFu, v0, 1), h1 = __shfl_sync(0xFFFFFFFFu, v1, 0);
            const float d1 = __shfl_down_sync(0xFFFFFFFFu, v1, 1);
            if (lane >= pos) v0 = (lane == 31) ? h1 : d0;
            if (lane + 32 >= pos) v1 = d1;
            --ns;
            dirty_from = min(dirty_from, pos);
        }
#pragma unroll
        for (int i = 0; i < NEW; ++i) {
            const float x = __shfl_sync(0xFFFFFFFFu, xe[i], src);
            if (!((me >> i) & 1u) || !good) continue;
            if (ns >= kIncSlots) { good = false; continue; }
            const uint32_t kx = f2key(x);
            // behind the listed values whose key is not above x's
            const int at = __popc(__ballot_sync(0xFFFFFFFFu, lane < ns && f2key(v0) <= kx)) +
                           __popc(__ballot_sync(0xFFFFFFFFu, lane + 32 < ns && f2key(v1) <= kx));
            const float u0 = __shfl_up_sync(0xFFFFFFFFu, v0, 1), t0 = __shfl_sync(0xFFFFFFFFu, v0, 31);
            const float u1 = __shfl_up_sync(0xFFFFFFFFu, v1, 1);
            if (lane + 32 > at) v1 = (lane == 0) ? t0 : u1;
            else if (lane + 32 == at) v1 = x;
            if (lane > at) v0 = u0;
            else if (lane == at) v0 = x;
            ++ns;
            dirty_from = min(dirty_from, at);
        }
        const int cbs = __shfl_sync(0xFFFFFFFFu, cb, src);
        good = good && cbs >= 0 && cbs <= k1 && k2 < cbs + ns;
        if (good) {   // write back the part that moved; hand the middle ranks' values to the series' own lane
            if (lane >= dirty_from && lane < ns) s.val[lbase + lane] = v0;
            if (lane + 32 >= dirty_from && lane + 32 < ns) s.val[lbase + lane + 32] = v1;
        }
        const int j1 = good ? k1 - cbs : 0, j2 = good ? k2 - cbs : 0;
        const float g10 = __shfl_sync(0xFFFFFFFFu, v0, j1 & 31), g11 = __shfl_sync(0xFFFFFFFFu, v1, j1 & 31);
        const float g20 = __shfl_sync(0xFFFFFFFFu, v0, j2 & 31), g21 = __shfl_sync(0xFFFFFFFFu, v1, j2 & 31);
        if (lane == src) {
            ok = good;
            nin = ns;
            f1 = (j1 >> 5) ? g11 : g10;
            f2 = (j2 >> 5) ? g21 : g20;
            have = true;
        }
    }
    ok = ok && cb >= 0 && cb <= k1 && k2 < cb + nin;
    if (ok) {
        // the list is sorted: the middle ranks of the window are positions k1 - cb and k2 - cb of it
        if (!have) {
            f1 = s.val[(size_t)c * kIncSlots + (k1 - cb)];
            f2 = s.val[(size_t)c * kIncSlots + (k2 - cb)];
        }
        const float med = median_from_keys(f2key(f1), f2key(f2), even);
        a.wmed[c] = med;
        if (a.wmed_user) a.wmed_user[c] = med;
        s.cnt[c] = 0x80000000u | ((uint32_t)nin << 16) | (uint32_t)cb;
    }
    // ---- series without a usable state go on the launch's rebuild list (window_rebuild_kernel follows) ----
    const unsigned todo = __ballot_sync(0xFFFFFFFFu, active && !ok);
    if (todo) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(s.rb_count, (uint32_t)__popc(todo));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if ((todo >> lane) & 1u) s.rb_list[base + __popc(todo & ((1u << lane) - 1u))] = (uint32_t)c;
    }
}

// The rebuilds of a launch, one warp per listed series (a few per thousand series in steady state, all of them
// when sliding starts): the lanes fetch the window, sort it (bitonic network over registers and shuffles), take
// the median, the interval ends kIncHalf ranks beyond the middle ranks, and the values inside.  A kernel of its
// own so that the rebuilds spread over the whole GPU instead of queueing inside the warps that found them.
constexpr int kRbThreads = 128;
constexpr int kRbCtas = 148 * 8;

template <int VPL>
__global__ void __launch_bounds__(kRbThreads) window_rebuild_kernel(const WindowArgs a, const IncArgs s) {
    __shared__ int is_last;
    const int lane = lane_id();
    const int n = a.n;
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;
    const bool even = !(n & 1);
    const int k1 = (n - 1) >> 1, k2 = n >> 1;
    const uint32_t count = min(__ldcg(s.rb_count), (uint32_t)a.series);
    const uint32_t nwarps = gridDim.x * (kRbThreads / 32);
    for (uint32_t i = blockIdx.x * (kRbThreads / 32) + warp_id(); i < count; i += nwarps) {
        const int series = (int)__ldcg(s.rb_list + i);
        uint32_t kv[VPL];
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int row = lane + 32 * j;
            kv[j] = 0xFFFFFFFFu;                 // padding sorts behind every finite value
            if (row < n) {
                int slot = first + row;
                if (slot >= a.capacity) slot -= a.capacity;
                kv[j] = f2key(__ldg(a.ring + (size_t)slot * a.row_stride + series));
            }
        }
        warp_bitonic_sort<VPL>(kv, lane);        // ascending: element e in lane e / VPL, register e % VPL
        auto pick = [&](int r) -> uint32_t {
            uint32_t mine = kv[0];
#pragma unroll
            for (int j = 1; j < VPL; ++j) mine = ((r % VPL) == j) ? kv[j] : mine;
            return __shfl_sync(0xFFFFFFFFu, mine, r / VPL);
        };
        const float med = median_from_keys(pick(k1), pick(k2), even);
        const float flo = key2f(pick(max(0, k1 - kIncHalf))), fhi = key2f(pick(min(n - 1, k2 + kIncHalf)));
        // values below / inside the interval, by the same float comparisons the sliding update uses
        int below = 0, in = 0;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const bool real = lane * VPL + j < n;
            const float x = key2f(kv[j]);
            below += real && (x < flo);
            in += real && !(x < flo) && (x <= fhi);
        }
        int incl = in;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int u = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += u;
        }
        const int nin2 = __shfl_sync(0xFFFFFFFFu, incl, 31);
        const int cb2 = (int)__reduce_add_sync(0xFFFFFFFFu, (uint32_t)below);
        const bool fits = nin2 <= kIncSlots;
        if (fits) {
            int pos = incl - in;
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const bool real = lane * VPL + j < n;
                const float x = key2f(kv[j]);
                if (real && !(x < flo) && (x <= fhi)) { s.val[(size_t)series * kIncSlots + pos] = x; ++pos; }
            }
        }
        if (lane == 0) {
            a.wmed[series] = med;
            if (a.wmed_user) a.wmed_user[series] = med;
            s.lo[series] = flo;
            s.hi[series] = fhi;
            // an interval with more (tied) values than a list holds stays without state: it rebuilds every time
            s.cnt[series] = fits ? (0x80000000u | ((uint32_t)nin2 << 16) | (uint32_t)cb2) : 0u;
            if (s.rebuilds) atomicAdd(s.rebuilds, 1u);
        }
    }
    // the CTA that finishes last clears the list for the next launch
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(s.rb_count + 1, 1u) == gridDim.x - 1u) ? 1 : 0;
    __syncthreads();
    if (is_last && threadIdx.x == 0) {
        s.rb_count[0] = 0u;
        s.rb_count[1] = 0u;
    }
}

// Fallback for windows too long to stage: one thread per series, bit-by-bit counting
// selection straight from global memory (32 sweeps of the column).
__global__ void window_select_global_kernel(const WindowArgs a) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= a.series) return;
    const int n = a.n;
    const int first = ((a.last_slot - (n - 1)) % a.capacity + a.capacity) % a.capacity;
    auto key_at = [&](int j) {
        int slot = first + j;
        if (slot >= a.capacity) slot -= a.capacity;
        return f2key(a.ring[(size_t)slot * a.row_stride + c]);
    };
    const int k = (n - 1) >> 1;
    uint32_t prefix = 0;
    int krem = k;
    for (int bit = 31; bit >= 0; --bit) {
        int zeros = 0;
        for (int j = 0; j < n; ++j) {
            const uint32_t key = key_at(j);
            const bool match = (bit == 31) || (((key ^ prefix) >> (bit + 1)) == 0);
            zeros += (match && !((key >> bit) & 1u));
        }
        if (krem >= zeros) {
            prefix |= 1u << bit;
            krem -= zeros;
        }
    }
    float med = key2f(prefix);
    if (!(n & 1)) {
        int cle = 0;
        uint32_t above = 0xFFFFFFFFu;
        for (int j = 0; j < n; ++j) {
            const uint32_t key = key_at(j);
            cle += (key <= prefix);
            if (key > prefix) above = min(above, key);
        }
        med = median_from_keys(prefix, cle > k + 1 ? prefix : above, true);
    }
    a.wmed[c] = med;
    if (a.wmed_user) a.wmed_user[c] = med;
}

template <int TC>
cudaError_t launch_staged(const WindowArgs &a, int use_bulk, cudaStream_t st) {
    const size_t smem = (size_t)a.n * TC * 4;
    static AttrOnce once;
    int dev = 0;
    cudaError_t e = once(dev, [] {
        return cudaFuncSetAttribute(window_select_kernel<TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxStagedTile);
    });
    if (e != cudaSuccess) return e;
    const int grid = (a.series + TC - 1) / TC;
    window_select_kernel<TC><<<grid, TC, smem, st>>>(a, use_bulk);
    return cudaGetLastError();
}

}  // namespace

int window_launch_count(const WindowArgs &a) { return (a.use_hint && a.spread && a.centre && a.fb_list && a.series < (1 << 28) && a.n <= 256) ? 2 : 1; }

size_t window_inc_bytes(int series) { return (size_t)series * sizeof(float); }

bool window_inc_supported(const WindowArgs &a) { return a.n >= 1 && a.n <= 256; }

cudaError_t launch_window_incremental(const WindowArgs &a, const IncArgs &inc, cudaStream_t st) {
    const int grid = (a.series + kIncThreads - 1) / kIncThreads;
    const int rgrid = min(kRbCtas, (a.series + kRbThreads / 32 - 1) / (kRbThreads / 32));
    if (inc.entering <= 1 && inc.leaving <= 1) window_inc_kernel<1><<<grid, kIncThreads, 0, st>>>(a, inc);
    else window_inc_kernel<kIncMaxNew><<<grid, kIncThreads, 0, st>>>(a, inc);
    if (a.n <= 64) window_rebuild_kernel<2><<<rgrid, kRbThreads, 0, st>>>(a, inc);
    else if (a.n <= 128) window_rebuild_kernel<4><<<rgrid, kRbThreads, 0, st>>>(a, inc);
    else window_rebuild_kernel<8><<<rgrid, kRbThreads, 0, st>>>(a, inc);
    return cudaGetLastError();
}

cudaError_t launch_window_select(const WindowArgs &a, cudaStream_t st) {
    constexpr size_t kMaxTile = kMaxStagedTile;
    // bulk copies need 16-byte aligned sources and sizes
    const int use_bulk = (a.series % 4 == 0) && (((uintptr_t)a.ring & 15) == 0);
    const size_t n = (size_t)a.n;
    if (a.use_hint && a.spread && a.centre && a.fb_list && a.series < (1 << 28) && n <= 256) {
        if (n <= 64) return launch_thread_path<2>(a, st);
        if (n <= 128) return launch_thread_path<4>(a, st);
        return launch_thread_path<8>(a, st);
    }
    if (n <= 64) return launch_warp_path<2>(a, use_bulk, st);
    if (n <= 128) return launch_warp_path<4>(a, use_bulk, st);
    if (n <= 256) return launch_warp_path<8>(a, use_bulk, st);
    if (n * 128 * 4 <= kMaxTile) return launch_staged<128>(a, use_bulk, st);
    if (n * 64 * 4 <= kMaxTile) return launch_staged<64>(a, use_bulk, st);
    if (n * 32 * 4 <= kMaxTile) return launch_staged<32>(a, use_bulk, st);
    const int threads = 128;
    window_select_global_kernel<<<(a.series + threads - 1) / threads, threads, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace guard
