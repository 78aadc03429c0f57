// Node-sweep qualification: per-GPU medians of repeated benchmark results, and the
// pass / fail verdicts against the fleet distribution (GPU level, then node level).
#include <math_constants.h>

#include "colselect.cuh"
#include "kernels.h"
#include "thselect.cuh"
#include "warpselect.cuh"

namespace guard {

namespace {

constexpr int kSweepCols = 128;

// One CTA stages the [reps][M] blocks of GT = 128 / M GPUs, transposed to one column per
// (GPU, metric) series, then every thread selects inside its own column.
__global__ void __launch_bounds__(kSweepCols) sweep_median_kernel(const SweepMedArgs a) {
    extern __shared__ __align__(16) uint32_t tile[];
    const int tid = threadIdx.x, M = a.M, reps = a.reps;
    const int gt = kSweepCols / M;
    const int g0 = blockIdx.x * gt;
    const int ng = min(gt, a.G - g0);
    const int per = reps * M;
    bool bad = false;
    for (int gl = 0; gl < ng; ++gl) {
        const float *src = a.S + (size_t)(g0 + gl) * per;
        for (int i = tid; i < per; i += kSweepCols) {
            const int rep = i / M, m = i - rep * M;
            const uint32_t b = __float_as_uint(src[i]);
            bad |= nonfinite_bits(b);
            tile[(size_t)rep * kSweepCols + gl * M + m] = key_of_bits(b);
        }
    }
    if (a.status && __any_sync(0xFFFFFFFFu, bad) && lane_id() == 0) atomicOr(a.status, kStatNonFinite);
    __syncthreads();
    if (tid >= ng * M) return;
    const float med = col_median(tile + tid, kSweepCols, reps);
    const size_t o = (size_t)g0 * M + tid;
    a.gmed[o] = med;
    if (a.gmed_user) a.gmed_user[o] = med;
}

// Warp-per-GPU path (up to 256 repetitions): the benchmark results of one GPU are one contiguous
// [reps][M] block, so a warp fetches its GPU's block with whole-line 128-bit loads into its slice
// of shared memory; then, metric by metric, the lanes pick the metric's column out of the block
// (VPL keys per lane), sort their own keys and run the warp selection.  Eight warps per CTA, a
// few kilobytes of shared memory per warp: every SM holds dozens of GPUs at once.
constexpr int kSweepWarps = 8;

template <int VPL>
__global__ void __launch_bounds__(kSweepWarps * 32) sweep_median_warp_kernel(const SweepMedArgs a) {
    extern __shared__ __align__(16) float sbuf[];      // [kSweepWarps][per], per rounded up to a multiple of 4
    const int lane = lane_id(), w = warp_id(), M = a.M, reps = a.reps;
    const int per = reps * M, per4 = (per + 3) & ~3;
    const int g = blockIdx.x * kSweepWarps + w;
    if (g >= a.G) return;                               // warps are independent: no CTA barrier below
    float *buf = sbuf + (size_t)w * per4;
    const float *src = a.S + (size_t)g * per;
    bool bad = false;
    if ((per & 3) == 0 && ((uintptr_t)a.S & 15) == 0) {
        for (int i = 4 * lane; i < per; i += 128) {
            const float4 v = __ldg(reinterpret_cast<const float4 *>(src + i));
            bad |= nonfinite_bits(__float_as_uint(v.x)) | nonfinite_bits(__float_as_uint(v.y)) |
                   nonfinite_bits(__float_as_uint(v.z)) | nonfinite_bits(__float_as_uint(v.w));
            *reinterpret_cast<float4 *>(buf + i) = v;
        }
    } else {
        for (int i = lane; i < per; i += 32) {
            const float v = __ldg(src + i);
            bad |= nonfinite_bits(__float_as_uint(v));
            buf[i] = v;
        }
    }
    if (a.status && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(a.status, kStatNonFinite);
    __syncwarp();
    for (int m = 0; m < M; ++m) {
        uint32_t kv[VPL];
        int nreal = 0;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int rep = lane + 32 * j;
            const bool real = rep < reps;
            kv[j] = real ? f2key(buf[rep * M + m]) : 0xFFFFFFFFu;
            nreal += real;
        }
        lane_sort<VPL>(kv);
        float med = 0.0f;
        const bool ok = warp_median<VPL>(kv, nreal, reps, 0u, med);
        if (lane == 0) {
            if (!ok && a.status) atomicOr(a.status, kStatInternal);
            const size_t o = (size_t)g * M + m;
            a.gmed[o] = med;
            if (a.gmed_user) a.gmed_user[o] = med;
        }
    }
}

template <int VPL>
cudaError_t launch_sweep_warp(const SweepMedArgs &a, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(sweep_median_warp_kernel<VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    sweep_median_warp_kernel<VPL><<<(a.G + kSweepWarps - 1) / kSweepWarps, kSweepWarps * 32, smem, st>>>(a);
    return cudaGetLastError();
}

// Thread-per-series path (32 to 256 repetitions): a series' repetitions scatter around their mean, and the
// mean predicts the median of 200 repetitions to a few hundredths of their standard deviation.  Pass A takes
// mean and standard deviation (the GPU's block is read once from HBM and stays in L1 / L2 for pass B); pass B
// counts the values below mean -/+ 0.2 sd and keeps those inside (about a sixth of them) in the thread's
// shared-memory column; the two middle ranks are then found among the kept keys (pivot search, as for the
// window medians).  A series whose
// counts do not prove the bracket (or whose column overflows) goes on a list for sweep_median_finish_kernel.
constexpr int kSwThreads = 128;
constexpr int kSwSlots = 60;      // kept keys per series (the column format of the thread-per-series selection)
constexpr int kSwRows = 8;        // repetitions in flight per thread
constexpr int kSwMaxPasses = 12;

__global__ void __launch_bounds__(kSwThreads) sweep_median_thread_kernel(const SweepMedArgs a) {
    __shared__ __align__(16) uint32_t kept[kSwThreads * kSwSlots];
    const int tid = threadIdx.x, M = a.M, n = a.reps;
    const long long series = (long long)a.G * M;
    const long long sidx = (long long)blockIdx.x * kSwThreads + tid;
    const bool active = sidx < series;
    const long long sc = active ? sidx : series - 1;
    const int g = (int)(sc / M), m = (int)(sc - (long long)g * M);
    const float *base = a.S + (size_t)g * n * M + m;

    // pass A: mean and variance about the first value (no cancellation for values far from zero); a series
    // whose repetitions all have the same bits is its own median
    const float x0 = __ldg(base);
    const uint32_t bits0 = __float_as_uint(x0);
    float sd1 = 0.0f, sd2 = 0.0f;
    bool bad = false, same = true;
    auto acc = [&](const float xv) {
        const uint32_t b = __float_as_uint(xv);
        bad |= nonfinite_bits(b);
        same = same && (b == bits0);
        const float d = xv - x0;
        sd1 += d;
        sd2 = fmaf(d, d, sd2);
    };
    int r = 0;
    for (; r + kSwRows <= n; r += kSwRows) {
        float x[kSwRows];
#pragma unroll
        for (int u = 0; u < kSwRows; ++u) x[u] = __ldg(base + (size_t)(r + u) * M);
#pragma unroll
        for (int u = 0; u < kSwRows; ++u) acc(x[u]);
    }
    for (; r < n; ++r) acc(__ldg(base + (size_t)r * M));
    if (a.status && __any_sync(0xFFFFFFFFu, bad && active) && lane_id() == 0) atomicOr(a.status, kStatNonFinite);
    const float inv = 1.0f / (float)n;
    const float mean_d = sd1 * inv;
    const float var = fmaxf(sd2 * inv - mean_d * mean_d, 0.0f);
    const float c = x0 + mean_d, h = 0.2f * sqrtf(var);
    const bool usable = active && !bad && !same && (h > 0.0f) && (h < 3.0e38f) && (fabsf(c) < 3.0e38f);
    float flo = c - h, fhi = c + h;
    if (flo == 0.0f) flo = -0.0f;   // an end that is zero admits both zeros: float compares then agree with the key order
    if (fhi == 0.0f) fhi = 0.0f;
    if (!usable) { flo = CUDART_INF_F; fhi = -CUDART_INF_F; }
    const uint32_t klo = usable ? f2key(flo) : 0xFFFFFFFFu, khi = usable ? f2key(fhi) : 0u;

    // pass B (the block is in L1 / L2 by now): count below, keep inside
    const uint32_t kbase = (uint32_t)__cvta_generic_to_shared(kept + tid * kSwSlots), klim = kbase + (uint32_t)(kSwSlots * 4);
    uint32_t kaddr = kbase, clt = 0;
    if (__any_sync(0xFFFFFFFFu, usable)) {
        r = 0;
        for (; r + kSwRows <= n; r += kSwRows) {
            float x[kSwRows];
#pragma unroll
            for (int u = 0; u < kSwRows; ++u) x[u] = __ldg(base + (size_t)(r + u) * M);
#pragma unroll
            for (int u = 0; u < kSwRows; ++u) th_cell(x[u], flo, fhi, klim, clt, kaddr);
        }
        for (; r < n; ++r) th_cell(__ldg(base + (size_t)r * M), flo, fhi, klim, clt, kaddr);
    }
    const bool even = !(n & 1);
    const int k1 = (n - 1) >> 1, k2 = n >> 1;
    const int nk = (int)((kaddr - kbase) >> 2);
    bool ok = usable && (int)clt <= k1 && k2 < (int)clt + nk && nk <= kSwSlots;
    uint32_t vb = 0, vu = 0;
    th_select_pair<kSwSlots, kSwMaxPasses>(kbase, nk, ok, k2 - (int)clt, klo, khi, vb, vu);
    float med = 0.0f;
    if (ok) med = median_from_keys(even ? vb : vu, vu, even);
    if (active && same && !bad) { med = x0; ok = true; }
    if (active && ok) {
        a.gmed[sidx] = med;
        if (a.gmed_user) a.gmed_user[sidx] = med;
    }
    const unsigned todo = __ballot_sync(0xFFFFFFFFu, active && !ok);
    if (todo) {
        const int lane = lane_id();
        uint32_t b = 0;
        if (lane == 0) b = atomicAdd(a.list_count, (uint32_t)__popc(todo));
        b = __shfl_sync(0xFFFFFFFFu, b, 0);
        if ((todo >> lane) & 1u) a.list[b + __popc(todo & ((1u << lane) - 1u))] = (uint32_t)sidx;
    }
}

// The listed series, one warp each: the lanes fetch the repetitions, sort their own keys and run the warp selection.
template <int VPL>
__global__ void __launch_bounds__(kSwThreads) sweep_median_finish_kernel(const SweepMedArgs a) {
    const int lane = lane_id(), M = a.M, n = a.reps;
    const uint32_t count = min(__ldcg(a.list_count), (uint32_t)min((long long)a.G * M, 0x7FFFFFFFLL));
    const uint32_t nwarps = gridDim.x * (kSwThreads / 32);
    for (uint32_t i = blockIdx.x * (kSwThreads / 32) + warp_id(); i < count; i += nwarps) {
        const uint32_t sidx = __ldcg(a.list + i);
        const int g = (int)(sidx / (uint32_t)M), m = (int)(sidx - (uint32_t)g * (uint32_t)M);
        const float *base = a.S + (size_t)g * n * M + m;
        uint32_t kv[VPL];
        int nreal = 0;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int rep = lane + 32 * j;
            const bool real = rep < n;
            kv[j] = real ? f2key(__ldg(base + (size_t)rep * M)) : 0xFFFFFFFFu;
            nreal += real;
        }
        lane_sort<VPL>(kv);
        float med = 0.0f;
        const bool ok = warp_median<VPL>(kv, nreal, n, 0u, med);
        if (lane == 0) {
            if (!ok && a.status) atomicOr(a.status, kStatInternal);
            a.gmed[sidx] = med;
            if (a.gmed_user) a.gmed_user[sidx] = med;
        }
    }
}

// Fallback when the repetitions of one GPU do not fit a tile: bit-by-bit counting
// selection from global memory, one thread per (GPU, metric).
__global__ void sweep_median_global_kernel(const SweepMedArgs a) {
    const long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= (long long)a.G * a.M) return;
    const int g = (int)(c / a.M), m = (int)(c - (long long)g * a.M);
    const float *src = a.S + (size_t)g * a.reps * a.M + m;
    const int n = a.reps, k = (n - 1) >> 1;
    uint32_t prefix = 0;
    int krem = k;
    bool bad = false;
    for (int bit = 31; bit >= 0; --bit) {
        int zeros = 0;
        for (int j = 0; j < n; ++j) {
            const uint32_t raw = __float_as_uint(src[(size_t)j * a.M]);
            bad |= nonfinite_bits(raw);
            const uint32_t key = key_of_bits(raw);
            const bool match = (bit == 31) || (((key ^ prefix) >> (bit + 1)) == 0);
            zeros += (match && !((key >> bit) & 1u));
        }
        if (krem >= zeros) {
            prefix |= 1u << bit;
            krem -= zeros;
        }
    }
    if (bad && a.status) atomicOr(a.status, kStatNonFinite);
    float med = key2f(prefix);
    if (!(n & 1)) {
        int cle = 0;
        uint32_t above = 0xFFFFFFFFu;
        for (int j = 0; j < n; ++j) {
            const uint32_t key = f2key(src[(size_t)j * a.M]);
            cle += (key <= prefix);
            if (key > prefix) above = min(above, key);
        }
        med = median_from_keys(prefix, cle > k + 1 ? prefix : above, true);
    }
    a.gmed[c] = med;
    if (a.gmed_user) a.gmed_user[c] = med;
}

// One thread per node: robust-z outlier AND beyond the percentile cut fails a metric;
// a GPU passes with no failed metric; a node passes when all of its GPUs pass.
__global__ void sweep_verdict_kernel(const SweepVerdictArgs a, const MetricParams p) {
    const int node = blockIdx.x * blockDim.x + threadIdx.x;
    if (node >= a.nodes) return;
    bool node_ok = true;
    for (int q = 0; q < a.gpus_per_node; ++q) {
        const size_t g = (size_t)node * a.gpus_per_node + q;
        uint32_t fail = 0;
        for (int m = 0; m < a.M; ++m) {
            const float v = a.gmed[g * a.M + m];
            const float F = a.fleet_med[m];
            const float Fs = scale_of(a.fleet_mad[m], F, p.floor_rel[m], p.floor_abs[m]);
            const bool zfail = exceeds(v, F, p.dir[m], __fmul_rn(p.thrp[m], Fs));
            const float cut = a.fleet_cut[m];
            const bool pfail = p.dir[m] < 0 ? (v < cut) : (v > cut);
            if (zfail && pfail) fail |= 1u << m;
        }
        if (a.fail_mask) a.fail_mask[g] = fail;
        if (a.gpu_pass) a.gpu_pass[g] = (uint8_t)(fail == 0);
        node_ok = node_ok && (fail == 0);
    }
    if (a.node_pass) a.node_pass[node] = (uint8_t)node_ok;
}

}  // namespace

cudaError_t launch_sweep_medians(const SweepMedArgs &a, cudaStream_t st) {
    const long long series = (long long)a.G * a.M;
    if (a.list && a.list_count && a.reps >= 32 && a.reps <= 256 && series < 0x7FFFFFFFLL) {
        cudaError_t e = cudaMemsetAsync(a.list_count, 0, sizeof(uint32_t), st);
        if (e != cudaSuccess) return e;
        sweep_median_thread_kernel<<<(unsigned)((series + kSwThreads - 1) / kSwThreads), kSwThreads, 0, st>>>(a);
        const long long want = (series + kSwThreads / 32 - 1) / (kSwThreads / 32);
        const int fgrid = (int)(want < 148 * 4 ? want : 148 * 4);
        if (a.reps <= 64) sweep_median_finish_kernel<2><<<fgrid, kSwThreads, 0, st>>>(a);
        else if (a.reps <= 128) sweep_median_finish_kernel<4><<<fgrid, kSwThreads, 0, st>>>(a);
        else sweep_median_finish_kernel<8><<<fgrid, kSwThreads, 0, st>>>(a);
        return cudaGetLastError();
    }
    const size_t wsmem = (size_t)kSweepWarps * (((size_t)a.reps * a.M + 3) & ~(size_t)3) * sizeof(float);
    if (a.reps <= 256 && wsmem <= 96 * 1024) {
        if (a.reps <= 64) return launch_sweep_warp<2>(a, wsmem, st);
        if (a.reps <= 128) return launch_sweep_warp<4>(a, wsmem, st);
        return launch_sweep_warp<8>(a, wsmem, st);
    }
    const size_t smem = (size_t)a.reps * kSweepCols * 4;
    if (smem <= 200 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(sweep_median_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const int gt = kSweepCols / a.M;
        sweep_median_kernel<<<(a.G + gt - 1) / gt, kSweepCols, smem, st>>>(a);
    } else {
        const long long series = (long long)a.G * a.M;
        sweep_median_global_kernel<<<(unsigned)((series + 127) / 128), 128, 0, st>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_sweep_verdict(const SweepVerdictArgs &a, const MetricParams &p, cudaStream_t st) {
    sweep_verdict_kernel<<<(a.nodes + 127) / 128, 128, 0, st>>>(a, p);
    return cudaGetLastError();
}

}  // namespace guard
