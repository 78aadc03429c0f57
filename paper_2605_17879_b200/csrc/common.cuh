// Shared declarations of the B200 straggler-scoring kernels: parameter block, status
// bits, the order-preserving key map and small warp helpers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace guard {

constexpr int kMaxMetrics = 32;
constexpr uint32_t kStatNonFinite = 1u;
constexpr uint32_t kStatTimeout = 2u;
constexpr uint32_t kStatInternal = 4u;

// Per-metric detector parameters, passed to kernels by value (no device copy needed).
struct MetricParams {
    int M;
    int primary;
    int min_signals;
    int n_consec;
    int k;
    float tier_moderate;
    float tier_severe;
    int8_t dir[kMaxMetrics];
    float thrp[kMaxMetrics];      // (float)(thr / 0.6745): cut-off moved to the right-hand side
    float floor_rel[kMaxMetrics];
    float floor_abs[kMaxMetrics];
};

// float32 -> uint32 such that the IEEE total order of finite floats is the unsigned
// order of the keys: negative values have all bits flipped, others only the sign bit.
__host__ __device__ __forceinline__ uint32_t key_of_bits(uint32_t b) {
    return b ^ ((b & 0x80000000u) ? 0xFFFFFFFFu : 0x80000000u);
}
__host__ __device__ __forceinline__ uint32_t bits_of_key(uint32_t k) {
    return k ^ ((k & 0x80000000u) ? 0x80000000u : 0xFFFFFFFFu);
}
__device__ __forceinline__ uint32_t f2key(float x) { return key_of_bits(__float_as_uint(x)); }
__device__ __forceinline__ float key2f(uint32_t k) { return __uint_as_float(bits_of_key(k)); }
__device__ __forceinline__ bool nonfinite_bits(uint32_t b) { return (b & 0x7F800000u) == 0x7F800000u; }

// Median of n values from the two middle order statistics (keys): lower middle for odd
// n (then lo == hi), midpoint with one add and one exact halving for even n.
__device__ __forceinline__ float median_from_keys(uint32_t klo, uint32_t khi, bool even) {
    float a = key2f(klo);
    if (!even) return a;
    return __fmul_rn(0.5f, __fadd_rn(a, key2f(khi)));
}

// Spread used by every robust-z test: the MAD floored relative to |median| and absolutely.
__device__ __forceinline__ float scale_of(float mad, float med, float floor_rel, float floor_abs) {
    float s = mad;
    float rel = __fmul_rn(floor_rel, fabsf(med));
    if (rel > s) s = rel;
    if (floor_abs > s) s = floor_abs;
    return s;
}

// One-sided exceedance in the metric's bad direction: dir * (x - med) > thrp * scale,
// with the right-hand side precomputed (rhs = thrp * scale).
__device__ __forceinline__ bool exceeds(float x, float med, int dir, float rhs) {
    float dev = __fsub_rn(x, med);
    if (dir < 0) dev = -dev;
    return dev > rhs;
}

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ int warp_id() { return threadIdx.x >> 5; }

}  // namespace guard
