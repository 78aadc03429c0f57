// Windowed per-series median: for every (rank, metric) series the exact median of its
// last n ring steps.  A CTA stages a [n steps] x [TC series] tile of the ring in shared
// memory with bulk asynchronous copies (one per ring row, completion on an mbarrier),
// then every thread selects inside its own column.
#include <math_constants.h>

#include <mutex>

#include "colselect.cuh"
#include "kernels.h"
#include "window_thread.cuh"

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
            const uint32_t hint = a.use_hint ? f2key(a.wmed[series]) : 0u;   // last evaluation's median
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

    th_finish<VPL>(a, first, c, active, usable, hint, h, klo, khi, kbase, kaddr, clt);
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
    return cudaGetLastError();
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

int window_launch_count(const WindowArgs &) { return 1; }

cudaError_t launch_window_select(const WindowArgs &a, cudaStream_t st) {
    constexpr size_t kMaxTile = kMaxStagedTile;
    // bulk copies need 16-byte aligned sources and sizes
    const int use_bulk = (a.series % 4 == 0) && (((uintptr_t)a.ring & 15) == 0);
    const size_t n = (size_t)a.n;
    if (a.use_hint && a.spread && a.centre && n <= 256) {
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
