// Tile kernels of the split cross-rank path: one CTA per tile of ranks, over ALL steps of the
// ingested block.
//
// A tile is 256 series wide (32 ranks x 8 metrics, or 64 ranks x 4): one step of it is 1 KiB of
// contiguous telemetry.  A producer warp stages the tile's rows, sixteen steps per stage, into a
// three-stage shared-memory ring with bulk asynchronous copies (TMA, one per row, completion counted
// on an mbarrier per stage); eight consumer warps read every staged value twice, in two
// orientations, so that the block crosses HBM once for both statistics:
//
//   cross-rank orientation (thread = one step of the stage, four metrics, four ranks): counts the
//     values below the step's sampled interval and notes which lie inside it.  The sixteen lanes of
//     a (step, metric quad) fold their counts with shuffles; one lane adds them to the step's packed
//     64-bit counters (four metrics per atomic) and, with a second atomic, reserves room for the
//     tile's kept elements in the four columns' lists.  The reservation's answer is needed only
//     after the window orientation has run, which hides its latency; then the kept values are
//     read from the stage again and stored.
//   window orientation (thread = one series, all steps; only in the median pass, when the block is
//     the window of the next evaluation): the one-thread-per-series count / keep step against the
//     series' own predicted interval; after the last stage every thread selects its median among
//     its kept keys (window_thread.cuh), so the windowed medians are ready when the block's
//     cross-rank statistics are.
//
// The MAD pass (MODE 1) is the same kernel on d = |x - med|, with the exceedance decisions of the
// rare large deviations taken inline, and no window orientation.
//
// Every wait has a time limit; a wait that runs out raises the sticky time-out status, the CTA lets
// the copies in flight land and leaves.
#include <mutex>

#include "window_thread.cuh"
#include "xsplit_common.cuh"

namespace guard {

namespace {

constexpr int kTlSeries = 256;                          // series per tile = consumer threads
constexpr int kTlSteps = 16;                            // steps per stage
constexpr int kTlStages = 3;
constexpr int kTlConsumerWarps = kTlSeries / 32;
constexpr int kTlThreads = kTlSeries + 32;              // consumers + the producer warp
constexpr int kTlRowBytes = kTlSeries * 4;
constexpr int kTlStageBytes = kTlSteps * kTlRowBytes;
constexpr int kTlListBytes = kTlSeries * kThSlots * 4;  // kept keys of the window orientation

struct TlShared {
    unsigned long long full[kTlStages], empty[kTlStages];
    int abort;
};

__device__ __forceinline__ bool tl_wait(uint64_t *bar, uint32_t parity, volatile int *abort) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort) return false;
        if (clock64() - t0 > kWaitLimitCycles) { *abort = 1; return false; }
    }
    return true;
}

__device__ __forceinline__ float4 tl_lds128(const uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float tl_lds32(const uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
// inclusive scan step inside each half-warp: v += value of lane (lane - d) when that lane is in the same 16-lane segment
__device__ __forceinline__ void tl_scan_step16(uint32_t &v, const int d) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 r;\n\tshfl.sync.up.b32 r|p, %0, %1, 0x1000, 0xffffffff;\n\t@p add.u32 %0, %0, r;\n\t}"
                 : "+r"(v)
                 : "r"(d));
}
// four 8-bit fields -> four 16-bit fields of a 64-bit word
__device__ __forceinline__ unsigned long long tl_widen(const uint32_t p8) {
    return (unsigned long long)__byte_perm(p8, 0, 0x4140) | ((unsigned long long)__byte_perm(p8, 0, 0x4342) << 32);
}

// NQ: float4 quads per rank (metrics / 4).  MODE 0: median pass, MODE 1: MAD / exceedance pass.
// WIN: the window orientation runs (MODE 0 only).
template <int NQ, int MODE, bool WIN>
__global__ void __launch_bounds__(kTlThreads, 2) xtile_kernel(const XrankArgs a, const MetricParams p, const SpScratch sc, const int S,
                                                             const WindowArgs w) {
    constexpr int M = 4 * NQ;
    constexpr int RT = kTlSeries / M;            // ranks per tile
    constexpr int G = 16 / NQ;                   // lanes of a (step, quad) group; each takes ranks g, g + G, g + 2 G, g + 3 G
    extern __shared__ __align__(128) unsigned char tl_smem[];
    __shared__ TlShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int R = a.R;
    const int r0 = blockIdx.x * RT;
    const int nranks = min(RT, R - r0);
    const uint32_t rowbytes = (uint32_t)nranks * M * 4u;
    const int nst = (S + kTlSteps - 1) / kTlSteps;
    const uint32_t stage0 = smem_u32(tl_smem);
    uint64_t *full = reinterpret_cast<uint64_t *>(sh.full), *empty = reinterpret_cast<uint64_t *>(sh.empty);
    volatile int *abortp = &sh.abort;

    if (tid == 0) {
        for (int i = 0; i < kTlStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], kTlConsumerWarps); }
        sh.abort = 0;
    }
    if (MODE == 1 && a.mask_base && tid < kTlSeries) {
        // this tile's part of every step's exceedance row starts at zero; bits are OR-ed in
        uint8_t *mb = reinterpret_cast<uint8_t *>(a.mask_base);
        const int words = nranks >> 2;          // ranks come in fours
        for (int i = tid; i < S * words; i += kTlSeries) {
            const int t = i / words, j = i - t * words;
            const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
            *reinterpret_cast<uint32_t *>(mb + (size_t)slot * R + r0 + 4 * j) = 0u;
        }
    }
    __syncthreads();

    int issued = 0;   // stages the producer has issued (meaningful in the producer warp)
    if (warp == kTlConsumerWarps) {
        // ---- producer ---------------------------------------------------------------------------
        for (int k = 0; k < nst; ++k) {
            const int s = k % kTlStages;
            if (k >= kTlStages && !__all_sync(0xFFFFFFFFu, tl_wait(&empty[s], (uint32_t)((k / kTlStages - 1) & 1), abortp))) break;
            const int rows = min(kTlSteps, S - k * kTlSteps);
            if (lane == 0) mbar_arrive_expect_tx(&full[s], (uint32_t)rows * rowbytes);
            __syncwarp();
            if (lane < rows) {
                const int t = k * kTlSteps + lane;
                const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
                bulk_g2s(tl_smem + (size_t)s * kTlStageBytes + (size_t)lane * kTlRowBytes,
                         a.base + (size_t)slot * a.row_stride + (size_t)r0 * M, rowbytes, &full[s]);
            }
            issued = k + 1;
        }
    } else {
        // ---- consumers --------------------------------------------------------------------------
        // window orientation: this thread's series
        const int c = r0 * M + tid;
        const bool active = WIN && tid < nranks * M;
        float hint = 0.0f, h = 0.0f, flo = CUDART_INF_F, fhi = -CUDART_INF_F;
        bool usable = false;
        uint32_t klo = 0xFFFFFFFFu, khi = 0u, clt = 0;
        const uint32_t kbase = stage0 + (uint32_t)(kTlStages * kTlStageBytes) + (uint32_t)tid * (uint32_t)(kThSlots * 4);
        const uint32_t klim = kbase + (uint32_t)(kThSlots * 4);
        uint32_t kaddr = kbase;
        const int w0 = WIN ? S - w.n : 0;       // first step of the block that belongs to the window
        if (WIN) {
            if (active) { hint = w.centre[c]; h = w.spread[c]; }
            usable = active && (h > 0.0f) && (h < 3.0e38f) && (fabsf(hint) < 3.0e38f);
            if (usable) {
                flo = hint - h; fhi = hint + h;
                if (flo == 0.0f) flo = -0.0f;
                if (fhi == 0.0f) fhi = 0.0f;
                klo = f2key(flo); khi = f2key(fhi);
            }
        }
        // cross-rank orientation: step sx of the stage, quad q, lane g of the group
        const int sx = tid >> 4, l16 = tid & 15, q = l16 & (NQ - 1), g = l16 / NQ;
        const uint32_t xoff = (uint32_t)sx * kTlRowBytes + (uint32_t)g * (M * 4) + (uint32_t)q * 16u;
        constexpr uint32_t kRankStride = (uint32_t)G * M * 4;   // bytes between this thread's consecutive ranks
        float sg[4], fr[4], fa[4];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
            sg[cc] = p.dir[4 * q + cc] < 0 ? -1.0f : 1.0f;
            fr[cc] = 0.0f; fa[cc] = 0.0f;
        }
        (void)fr; (void)fa;
        uint8_t *maskbase = reinterpret_cast<uint8_t *>(a.mask_base);
        const float *blo = MODE == 0 ? sc.blo : sc.bdlo, *bhi = MODE == 0 ? sc.bhi : sc.bdhi;

        for (int k = 0; k < nst; ++k) {
            const int s = k % kTlStages;
            const int rows = min(kTlSteps, S - k * kTlSteps);
            const int t = k * kTlSteps + sx;
            // the step's intervals come from global scratch (cached): issue the loads before the wait
            const bool xlive = sx < rows && sc.fail[min(t, S - 1)] == 0;
            float lo[4] = {0, 0, 0, 0}, hi[4] = {0, 0, 0, 0}, nsm[4] = {0, 0, 0, 0}, rlo[4] = {0, 0, 0, 0};
            if (xlive) {
                const float4 l4 = __ldg(reinterpret_cast<const float4 *>(blo + (size_t)t * M) + q);
                const float4 h4 = __ldg(reinterpret_cast<const float4 *>(bhi + (size_t)t * M) + q);
                lo[0] = l4.x; lo[1] = l4.y; lo[2] = l4.z; lo[3] = l4.w;
                hi[0] = h4.x; hi[1] = h4.y; hi[2] = h4.z; hi[3] = h4.w;
                if (MODE == 1) {
                    const float4 m4 = __ldg(reinterpret_cast<const float4 *>(sc.bmed + (size_t)t * M) + q);
                    const float4 r4 = __ldg(reinterpret_cast<const float4 *>(sc.brlo + (size_t)t * M) + q);
                    nsm[0] = -sg[0] * m4.x; nsm[1] = -sg[1] * m4.y; nsm[2] = -sg[2] * m4.z; nsm[3] = -sg[3] * m4.w;
                    rlo[0] = r4.x; rlo[1] = r4.y; rlo[2] = r4.z; rlo[3] = r4.w;
                }
            }
            if (!__all_sync(0xFFFFFFFFu, tl_wait(&full[s], (uint32_t)((k / kTlStages) & 1), abortp))) break;   // the warp decides as one
            const uint32_t sbase = stage0 + (uint32_t)s * kTlStageBytes;

            // ---- cross-rank orientation, part 1: count, note, reserve ---------------------------
            uint32_t cnt[4] = {0, 0, 0, 0}, inmask = 0;
            if (xlive) {
                float4 xv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) xv[i] = tl_lds128(sbase + xoff + (uint32_t)i * kRankStride);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const bool valid = g + i * G < nranks;
                    float v[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w};
                    if (MODE == 1) {
                        float sdev[4];
                        bool slow = false;
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            sdev[cc] = __fmaf_rn(v[cc], sg[cc], nsm[cc]);   // sign * (x - med), one rounding
                            v[cc] = fabsf(sdev[cc]);
                            slow |= !(v[cc] <= rlo[cc]);                    // beyond the threshold's lowest possible value, or not a number
                        }
                        if (slow && valid) {
                            // rare: the finite check, then exact tests against the threshold's possible range;
                            // the bit is set at once, or the decision is deferred until the MAD is known
                            const int r = r0 + g + i * G;
                            const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
                            uint32_t eb = 0;
#pragma unroll
                            for (int cc = 0; cc < 4; ++cc) {
                                const int m = 4 * q + cc;
                                const float xr = cc == 0 ? xv[i].x : cc == 1 ? xv[i].y : cc == 2 ? xv[i].z : xv[i].w;
                                if (a.check_finite && nonfinite_bits(__float_as_uint(xr))) atomicOr(a.status, kStatNonFinite);
                                if (sdev[cc] > rlo[cc]) {
                                    if (sdev[cc] > sc.col[(size_t)t * M + m].rhi) {
                                        eb |= 1u << m;
                                    } else {
                                        const uint32_t pos = atomicAdd(sc.namb + t, 1u);
                                        if (pos < (uint32_t)kSpAmb) sc.amb[(size_t)t * kSpAmb + pos] = ((uint32_t)r << 5) | (uint32_t)m;
                                    }
                                }
                            }
                            if (eb && maskbase)
                                atomicOr(reinterpret_cast<unsigned int *>(maskbase + (size_t)slot * R + (r & ~3)), eb << (8 * (r & 3)));
                        }
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const bool ge = v[cc] >= lo[cc];
                        const bool in = ge && (v[cc] <= hi[cc]) && valid;
                        cnt[cc] += (!ge && valid) ? 1u : 0u;
                        inmask |= in ? (1u << (4 * i + cc)) : 0u;
                    }
                }
            }
            // fold over the group's lanes: counts below (sum) and kept counts (inclusive scan), 8 bits per metric
            uint32_t cntp = cnt[0] | (cnt[1] << 8) | (cnt[2] << 16) | (cnt[3] << 24);
            const uint32_t keptp = (uint32_t)__popc(inmask & 0x1111u) | ((uint32_t)__popc(inmask & 0x2222u) << 8) |
                                   ((uint32_t)__popc(inmask & 0x4444u) << 16) | ((uint32_t)__popc(inmask & 0x8888u) << 24);
            uint32_t incl = keptp;
#pragma unroll
            for (int d = NQ; d < 16; d <<= 1) {
                cntp += __shfl_xor_sync(0xFFFFFFFFu, cntp, d);
                tl_scan_step16(incl, d);
            }
            const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, (lane & 16) | (16 - NQ + q));
            unsigned long long base64 = 0;
            if (g == 0 && xlive) {
                if (cntp) atomicAdd(sc.cnt64 + ((size_t)MODE * S + t) * NQ + q, tl_widen(cntp));
                if (total) base64 = atomicAdd(sc.nk64 + ((size_t)MODE * S + t) * NQ + q, tl_widen(total));
            }

            // ---- window orientation -------------------------------------------------------------
            if (WIN) {
                const int jlo = max(0, w0 - k * kTlSteps);
                const uint32_t wbase = sbase + (uint32_t)tid * 4u;
                if (jlo == 0 && rows == kTlSteps) {
                    float x[kTlSteps];
#pragma unroll
                    for (int j = 0; j < kTlSteps; ++j) x[j] = tl_lds32(wbase + (uint32_t)j * kTlRowBytes);
#pragma unroll
                    for (int j = 0; j < kTlSteps; ++j) th_cell(x[j], flo, fhi, klim, clt, kaddr);
                } else {
                    for (int j = jlo; j < rows; ++j) th_cell(tl_lds32(wbase + (uint32_t)j * kTlRowBytes), flo, fhi, klim, clt, kaddr);
                }
            }

            // ---- cross-rank orientation, part 2: store the kept values ----------------------------
            {
                const int src = (lane & 16) | q;   // the group's lane with g == 0
                const uint32_t blo32 = __shfl_sync(0xFFFFFFFFu, (uint32_t)base64, src);
                const uint32_t bhi32 = __shfl_sync(0xFFFFFFFFu, (uint32_t)(base64 >> 32), src);
                uint32_t run = incl - keptp;       // exclusive prefix of this lane, 8 bits per metric
                uint32_t mleft = inmask;
                while (mleft) {
                    const int b = __ffs(mleft) - 1;
                    mleft &= mleft - 1;
                    const int i = b >> 2, cc = b & 3;
                    float x = tl_lds32(sbase + xoff + (uint32_t)i * kRankStride + (uint32_t)cc * 4u);
                    if (MODE == 1) {
                        const float sgc = cc == 0 ? sg[0] : cc == 1 ? sg[1] : cc == 2 ? sg[2] : sg[3];
                        const float nsc = cc == 0 ? nsm[0] : cc == 1 ? nsm[1] : cc == 2 ? nsm[2] : nsm[3];
                        x = fabsf(__fmaf_rn(x, sgc, nsc));
                    }
                    const uint32_t bsel = (cc & 2) ? bhi32 : blo32;
                    const uint32_t pos = ((bsel >> (16 * (cc & 1))) & 0xFFFFu) + ((run >> (8 * cc)) & 0xFFu);
                    run += 1u << (8 * cc);
                    if (pos < (uint32_t)kTileCap) sc.clist[((size_t)t * M + 4 * q + cc) * kTileCap + pos] = __float_as_uint(x);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }

        if (WIN && !*abortp) {
            // nothing below waits on another warp: every consumer warp finishes its 32 series by itself
            const int first = (int)(((long long)a.first_slot + w0) % a.capacity);
            th_finish<8>(w, first, c, active, usable, hint, h, klo, khi, kbase, kaddr, clt);
        }
    }

    // ---- a wait ran out somewhere: report it, let the copies in flight land, leave ---------------
    __syncthreads();
    if (sh.abort) {
        if (tid == 0) atomicOr(a.status, kStatTimeout);
        if (warp == kTlConsumerWarps && lane == 0) {
            for (int k = max(0, issued - kTlStages); k < issued; ++k)
                mbar_wait_bounded(&full[k % kTlStages], (uint32_t)((k / kTlStages) & 1), kWaitLimitCycles);
        }
        __syncthreads();
    }
}

size_t tile_smem(bool win) { return (size_t)kTlStages * kTlStageBytes + (win ? kTlListBytes : 0); }

template <int NQ, int MODE, bool WIN>
cudaError_t launch_one(const XrankArgs &a, const MetricParams &p, const SpScratch &sc, int S, const WindowArgs &w, cudaStream_t st) {
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev & 63]) {
            e = cudaFuncSetAttribute(xtile_kernel<NQ, MODE, WIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tile_smem(WIN));
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(xtile_kernel<NQ, MODE, WIN>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
            done[dev & 63] = true;
        }
    }
    constexpr int RT = kTlSeries / (4 * NQ);
    const int tiles = (a.R + RT - 1) / RT;
    xtile_kernel<NQ, MODE, WIN><<<tiles, kTlThreads, tile_smem(WIN), st>>>(a, p, sc, S, w);
    return cudaGetLastError();
}

}  // namespace

bool xrank_tile_supported(int R, int M, int S) {
    // lists of kTileCap elements per column hold the ~10 % of a column the sampled intervals keep
    return (M == 4 || M == 8) && (R & 3) == 0 && R >= 4096 && R <= 20000 && S >= 1;
}

cudaError_t launch_xtile_sweep(int mode, const XrankArgs &a, const MetricParams &p, const SpScratch &sc, int S,
                               const TileWindow &win, cudaStream_t st) {
    WindowArgs w{};
    const bool fuse = mode == 0 && win.enabled;
    if (fuse) {
        w.ring = a.base;
        w.row_stride = a.row_stride;
        w.capacity = a.capacity;
        w.last_slot = (int)(((long long)a.first_slot + S - 1) % a.capacity);
        w.n = win.n;
        w.series = a.R * a.M;
        w.wmed = win.wmed;
        w.wmed_user = nullptr;
        w.use_hint = 1;
        w.spread = win.spread;
        w.centre = win.centre;
        w.target = win.target;
        w.smooth = win.smooth;
        w.fb_count = win.fb_count;
        w.status = a.status;
    }
    if (a.M == 8) {
        if (mode == 1) return launch_one<2, 1, false>(a, p, sc, S, w, st);
        return fuse ? launch_one<2, 0, true>(a, p, sc, S, w, st) : launch_one<2, 0, false>(a, p, sc, S, w, st);
    }
    if (mode == 1) return launch_one<1, 1, false>(a, p, sc, S, w, st);
    return fuse ? launch_one<1, 0, true>(a, p, sc, S, w, st) : launch_one<1, 0, false>(a, p, sc, S, w, st);
}

}  // namespace guard
