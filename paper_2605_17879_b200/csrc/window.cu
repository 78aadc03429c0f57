// Windowed per-series median: for every (rank, metric) series the exact median of its
// last n ring steps.  A CTA stages a [n steps] x [TC series] tile of the ring in shared
// memory with bulk asynchronous copies (one per ring row, completion on an mbarrier),
// then every thread selects inside its own column.
#include "colselect.cuh"
#include "kernels.h"

namespace guard {

namespace {

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
    for (int j = 0; j < n; ++j) col[(size_t)j * TC] = key_of_bits(col[(size_t)j * TC]);
    const float med = col_median(col, TC, n);
    a.wmed[col0 + tid] = med;
    if (a.wmed_user) a.wmed_user[col0 + tid] = med;
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
    cudaError_t e = cudaFuncSetAttribute(window_select_kernel<TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int grid = (a.series + TC - 1) / TC;
    window_select_kernel<TC><<<grid, TC, smem, st>>>(a, use_bulk);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_window_select(const WindowArgs &a, cudaStream_t st) {
    constexpr size_t kMaxTile = 200 * 1024;
    // bulk copies need 16-byte aligned sources and sizes
    const int use_bulk = (a.series % 4 == 0) && (((uintptr_t)a.ring & 15) == 0);
    const size_t n = (size_t)a.n;
    if (n * 128 * 4 <= kMaxTile) return launch_staged<128>(a, use_bulk, st);
    if (n * 64 * 4 <= kMaxTile) return launch_staged<64>(a, use_bulk, st);
    if (n * 32 * 4 <= kMaxTile) return launch_staged<32>(a, use_bulk, st);
    const int threads = 128;
    window_select_global_kernel<<<(a.series + threads - 1) / threads, threads, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace guard
