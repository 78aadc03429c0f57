// Node-sweep qualification: per-GPU medians of repeated benchmark results, and the
// pass / fail verdicts against the fleet distribution (GPU level, then node level).
#include "colselect.cuh"
#include "kernels.h"

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
