// Node-sweep qualification: per-GPU medians of repeated benchmark results, and the
// pass / fail verdicts against the fleet distribution (GPU level, then node level).
#include "colselect.cuh"
#include "kernels.h"
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
