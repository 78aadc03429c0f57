// Per-thread exact selection inside a strided shared-memory column, and the bulk-copy
// (TMA) / mbarrier primitives used to stage the tiles those columns live in.
#pragma once
#include "common.cuh"

namespace guard {

// ---- selection ------------------------------------------------------------------------

// k-th smallest (0-based) of col[0], col[stride], ..., col[(n-1)*stride] (uint32 keys).
// Three-way partitioning around a median-of-three pivot; the column is permuted in
// place (its multiset is preserved).  Each thread owns its column, so no barrier is
// needed; with one column per lane and a row pitch that is a multiple of 32 words every
// access of a warp is free of bank conflicts.  Loads are issued in batches of eight before
// the dependent compare / swap work, so that a thread keeps several shared-memory loads in
// flight (few warps fit next to the tiles, latency has to be hidden inside the thread).
// On return *below_end is the first position not known to hold a key < the result: every
// position before it holds a key <= the result.
constexpr int kSelBatch = 8;

__device__ __forceinline__ uint32_t col_select(uint32_t *col, int stride, int n, int k, int *below_end) {
    int l = 0, r = n - 1;
    while (l < r) {
        const uint32_t a = col[(size_t)l * stride], b = col[(size_t)((l + r) >> 1) * stride],
                       c = col[(size_t)r * stride];
        const uint32_t p = max(min(a, b), min(max(a, b), c));
        int store = l, ceq = 0;
        for (int i = l; i <= r; i += kSelBatch) {
            uint32_t v[kSelBatch];
#pragma unroll
            for (int u = 0; u < kSelBatch; ++u) v[u] = (i + u <= r) ? col[(size_t)(i + u) * stride] : 0xFFFFFFFFu;
#pragma unroll
            for (int u = 0; u < kSelBatch; ++u) {
                if (i + u <= r) {
                    if (v[u] < p) {   // earlier swaps of this batch never touch position i + u
                        col[(size_t)(i + u) * stride] = col[(size_t)store * stride];
                        col[(size_t)store * stride] = v[u];
                        ++store;
                    }
                    ceq += (v[u] == p);
                }
            }
        }
        if (k < store) {
            r = store - 1;
        } else if (k < store + ceq) {
            *below_end = store;
            return p;
        } else {
            int s2 = store;
            for (int i = store; i <= r; ++i) {
                const uint32_t v = col[(size_t)i * stride];
                if (v == p) {
                    col[(size_t)i * stride] = col[(size_t)s2 * stride];
                    col[(size_t)s2 * stride] = v;
                    ++s2;
                }
            }
            l = s2;
        }
    }
    *below_end = l;
    return col[(size_t)l * stride];
}

// Keys of ranks k - 1 (if want_prev) and k of a column.  Rank k is selected; rank k - 1 is then
// the same key if a further copy of it sits before position k, else the largest key among the
// positions the partitioning left before it.
__device__ __forceinline__ void col_rank_pair(uint32_t *col, int stride, int n, int k, bool want_prev, uint32_t &v_prev,
                                              uint32_t &v_k) {
    int below_end;
    v_k = col_select(col, stride, n, k, &below_end);
    v_prev = v_k;
    if (want_prev && below_end >= k) {
        uint32_t m = 0;
        for (int i = 0; i < below_end; i += kSelBatch) {
            uint32_t v[kSelBatch];
#pragma unroll
            for (int u = 0; u < kSelBatch; ++u) v[u] = (i + u < below_end) ? col[(size_t)(i + u) * stride] : 0u;
#pragma unroll
            for (int u = 0; u < kSelBatch; ++u) m = max(m, v[u]);
        }
        v_prev = m;
    }
}

// Median of a column of keys (midpoint rule for even n): ranks n/2 - 1 and n/2, or the middle.
__device__ __forceinline__ float col_median(uint32_t *col, int stride, int n) {
    uint32_t v1, v2;
    col_rank_pair(col, stride, n, n >> 1, !(n & 1), v1, v2);
    return median_from_keys(v1, v2, !(n & 1));
}

// ---- bulk async copy (TMA) + mbarrier ---------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Non-blocking probe of the phase (try_wait may suspend the thread for a while before it answers).
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
constexpr long long kShortWaitCycles = 100000;   // limits below this poll without suspending
// Waits for the phase with a time limit (in clock cycles); false if it ran out.  Short limits
// (test hooks) poll with the non-blocking probe, so that the limit and nothing else ends the wait.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, long long limit_cycles) {
    const long long t0 = clock64();
    if (limit_cycles < kShortWaitCycles) {
        while (!mbar_test_wait(bar, parity)) {
            if (clock64() - t0 > limit_cycles) return false;
        }
        return true;
    }
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit_cycles) return false;
    }
    return true;
}
// 1-D bulk copy global -> shared, completion counted in bytes on the mbarrier.  Both
// addresses and the size must be multiples of 16 bytes.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

constexpr long long kWaitLimitCycles = 2000000000LL;  // about one second

}  // namespace guard
