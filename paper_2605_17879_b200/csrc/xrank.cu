// Cross-rank selection: exact median and MAD of every (step, metric) column of a
// [steps][ranks][metrics] float32 array, plus the per-rank exceedance bits.
//
// Direct path: one CTA per step.  Values are mapped to order-preserving uint32 keys and
// the wanted order statistic is found by an 8-bit most-significant-digit radix select:
// four sweeps over the row, each filling one 256-bin shared-memory histogram per metric.
// Telemetry is tightly concentrated, so the leading digits of a column are almost
// constant; lanes that hit the same bin are therefore merged with __match_any_sync and
// only one lane per group issues the shared-memory atomic.
#include "xrank_direct.cuh"

namespace guard {

namespace {

constexpr int kXrThreads = 512;

__global__ void __launch_bounds__(kXrThreads) xrank_direct_kernel(const XrankArgs a, const MetricParams p) {
    extern __shared__ uint32_t hist[];
    __shared__ XrShared sh;
    const int s = blockIdx.x, tid = threadIdx.x;
    if (a.only_flagged && a.only_flagged[s] == 0) return;
    xrank_direct_step(a, p, s, hist, sh);
    if (a.only_flagged && tid == 0) {
        a.only_flagged[s] = 0;
        if (a.fallbacks) atomicAdd(a.fallbacks, 1u);
    }
}

}  // namespace

cudaError_t launch_xrank_direct(const XrankArgs &a, const MetricParams &p, int S, cudaStream_t st) {
    if (S <= 0) return cudaSuccess;
    const size_t smem = (size_t)a.M * 256 * sizeof(uint32_t);
    xrank_direct_kernel<<<S, kXrThreads, smem, st>>>(a, p);
    return cudaGetLastError();
}

}  // namespace guard
