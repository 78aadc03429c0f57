// Top-k slowest ranks, block then grid: every CTA keeps the best entries of its slice of
// ranks with a shared-memory bitonic network, writes its K best to scratch, and the CTA
// that takes the last ticket merges the per-CTA lists.  No CTA ever waits for another.
#include "kernels.h"

namespace guard {

namespace {

constexpr int kTopThreads = 1024;
constexpr int kTopChunk = 2048;  // entries merged into the running list at a time

// Sorts buf[0 .. 2 * kTopChunk) in descending order (all threads of the CTA).
__device__ void bitonic_desc(unsigned long long *buf) {
    constexpr int N = 2 * kTopChunk;
    for (int size = 2; size <= N; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < N / 2; t += blockDim.x) {
                const int i = 2 * t - (t & (stride - 1));
                const int j = i + stride;
                const bool desc = ((i & size) == 0);
                const unsigned long long x = buf[i], y = buf[j];
                if ((x < y) == desc) {
                    buf[i] = y;
                    buf[j] = x;
                }
            }
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kTopThreads) topk_kernel(const TopkArgs a, const MetricParams p, const int nblocks) {
    __shared__ unsigned long long buf[2 * kTopChunk];
    __shared__ int is_last;
    const int tid = threadIdx.x, b = blockIdx.x;
    const int pm = p.primary, dirp = p.dir[pm];
    const int per = (a.R + nblocks - 1) / nblocks;
    const int lo = b * per, hi = min(a.R, lo + per);

    for (int i = tid; i < kTopChunk; i += blockDim.x) buf[i] = 0ull;
    for (int c0 = lo; c0 < hi; c0 += kTopChunk) {
        for (int i = tid; i < kTopChunk; i += blockDim.x) {
            const int r = c0 + i;
            unsigned long long e = 0ull;
            if (r < hi) {
                float v = a.wmed[(size_t)r * a.M + pm];
                if (dirp < 0) v = -v;
                e = ((unsigned long long)f2key(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)r);
            }
            buf[kTopChunk + i] = e;
        }
        bitonic_desc(buf);
    }
    __syncthreads();
    if (nblocks > 1) {
        for (int i = tid; i < a.K; i += blockDim.x) a.cand[(size_t)b * a.K + i] = buf[i];
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned prev = atomicAdd(a.ticket, 1u);
            is_last = (prev == (unsigned)nblocks - 1u);
            if (is_last) *a.ticket = 0u;  // ready for the next launch
        }
        __syncthreads();
        if (!is_last) return;
        __threadfence();
        const int total = nblocks * a.K;
        for (int i = tid; i < kTopChunk; i += blockDim.x) buf[i] = 0ull;
        for (int c0 = 0; c0 < total; c0 += kTopChunk) {
            for (int i = tid; i < kTopChunk; i += blockDim.x)
                buf[kTopChunk + i] = (c0 + i < total) ? a.cand[c0 + i] : 0ull;
            bitonic_desc(buf);
        }
        __syncthreads();
    }
    const float B = a.fleet_med[pm];
    const float Ds = scale_of(a.fleet_mad[pm], B, p.floor_rel[pm], p.floor_abs[pm]);
    for (int i = tid; i < a.K; i += blockDim.x) {
        const int r = (int)(0xFFFFFFFFu - (uint32_t)(buf[i] & 0xFFFFFFFFull));
        if (a.idx) a.idx[i] = r;
        if (a.score) {
            float dev = __fsub_rn(a.wmed[(size_t)r * a.M + pm], B);
            if (dirp < 0) dev = -dev;
            a.score[i] = (dev == 0.0f) ? 0.0f : __fdiv_rn(__fmul_rn(0.6745f, dev), Ds);
        }
    }
}

}  // namespace

int topk_blocks(int R) {
    int nb = (R + kTopChunk - 1) / kTopChunk;
    return nb < 1 ? 1 : (nb > 64 ? 64 : nb);
}

cudaError_t launch_topk(const TopkArgs &a, const MetricParams &p, cudaStream_t st) {
    if (a.K <= 0 || (!a.idx && !a.score)) return cudaSuccess;
    const int nb = topk_blocks(a.R);
    topk_kernel<<<nb, kTopThreads, 0, st>>>(a, p, nb);
    return cudaGetLastError();
}

}  // namespace guard
