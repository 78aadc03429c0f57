// Top-k slowest ranks, block then grid: every CTA finds the K best entries of its slice of
// ranks (K-th largest key by histogram refinement in registers, then a small shared-memory
// bitonic sort of the entries at or above it), writes them to scratch, and the CTA that takes
// the last ticket folds the per-CTA lists the same way.  No CTA ever waits for another.
#include <cstdio>
#include <mutex>

#include "../../include/guard_b200.h"
#include "colreg.cuh"
#include "kernels.h"

namespace guard {

namespace {

constexpr int kTopThreads = 1024;
constexpr int kTopChunk = 1024;                 // ranks folded into the running list at a time
constexpr int kTopList = kTopChunk + 1024;      // a chunk plus the running list

// Sorts buf[0 .. n2) in descending order (n2 a power of two; all threads of the CTA).
__device__ void bitonic_desc(unsigned long long *buf, int n2) {
    for (int size = 2; size <= n2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < n2 / 2; t += blockDim.x) {
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

// Folds up to two entries per thread (64-bit composites: key of the value in the high
// word, ~rank in the low word; 0 = no entry) into the K best, left sorted in run[0..K).
// The K-th largest key is found by histogram refinement in registers; only the entries at
// or above it (K of them, plus ties) are sorted.
__device__ void fold_topk(const unsigned long long (&e)[2], int K, unsigned long long *list, unsigned long long *run,
                          ColShared &sh, uint32_t *s_n) {
    const int tid = threadIdx.x;
    uint32_t key[2];
    uint32_t valid = 0;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        key[i] = (uint32_t)(e[i] >> 32);
        if (e[i] != 0ull) valid |= 1u << i;
    }
    if (tid == 0) *s_n = 0;
    __syncthreads();
    const uint32_t mine = __popc(valid);
    const uint32_t wsum = __reduce_add_sync(0xFFFFFFFFu, mine);
    if (lane_id() == 0 && wsum) atomicAdd(s_n, wsum);
    __syncthreads();
    const uint32_t n = *s_n;
    __syncthreads();
    uint32_t thr = 0, dummy;
    if (n > (uint32_t)K) {
        if (!col_select_regs<2>(key, valid, n - (uint32_t)K, false, sh, thr, dummy)) thr = 0;
    }
    if (tid == 0) *s_n = 0;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 2; ++i)
        if (((valid >> i) & 1u) && key[i] >= thr) list[atomicAdd(s_n, 1u)] = e[i];
    __syncthreads();
    const int cnt = (int)*s_n;
    int n2 = 2;
    while (n2 < cnt) n2 <<= 1;
    for (int i = cnt + tid; i < n2; i += blockDim.x) list[i] = 0ull;
    bitonic_desc(list, n2);
    for (int i = tid; i < K; i += blockDim.x) run[i] = i < cnt ? list[i] : 0ull;
    __syncthreads();
}

__global__ void __launch_bounds__(kTopThreads) topk_kernel(const TopkArgs a, const MetricParams p, const int nblocks) {
    __shared__ unsigned long long list[kTopList];
    __shared__ unsigned long long run[2 * GUARD_MAX_TOPK];
    __shared__ ColShared sh;
    __shared__ uint32_t s_n;
    __shared__ int is_last;
    const int tid = threadIdx.x, b = blockIdx.x;
    if (a.hint && __ldcg(&a.hint->need_full) == 0) return;   // the hinted kernel in front has produced the list
    const int pm = p.primary, dirp = p.dir[pm];
    const int per = (a.R + nblocks - 1) / nblocks;
    const int lo = b * per, hi = min(a.R, lo + per);
    const int K = a.K;

    for (int i = tid; i < K; i += blockDim.x) run[i] = 0ull;
    __syncthreads();
    for (int c0 = lo; c0 < hi; c0 += kTopChunk) {
        unsigned long long e[2];
        const int r = c0 + tid;
        e[0] = 0ull;
        if (r < hi) {
            float v = a.wmed[(size_t)r * a.M + pm];
            if (dirp < 0) v = -v;
            e[0] = ((unsigned long long)f2key(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)r);
        }
        e[1] = tid < K ? run[tid] : 0ull;
        __syncthreads();
        fold_topk(e, K, list, run, sh, &s_n);
    }
    if (nblocks > 1) {
        for (int i = tid; i < K; i += blockDim.x) a.cand[(size_t)b * K + i] = run[i];
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
        const int total = nblocks * K;
        // with a hint state the fold keeps up to three times K entries: the last of them bounds the next
        // evaluation's threshold from below (at least that many ranks lie at or above it)
        const int K2 = a.hint ? min(3 * K, 2 * GUARD_MAX_TOPK) : K;
        for (int i = tid; i < K2; i += blockDim.x) run[i] = 0ull;
        __syncthreads();
        for (int c0 = 0; c0 < total; c0 += kTopChunk) {
            unsigned long long e[2];
            const int j = c0 + tid;
            e[0] = j < total ? __ldcg(a.cand + j) : 0ull;
            e[1] = tid < K2 ? run[tid] : 0ull;
            __syncthreads();
            fold_topk(e, K2, list, run, sh, &s_n);
        }
        if (a.hint && tid == 0) {
            int last = K2 - 1;
            while (last > 0 && run[last] == 0ull) --last;
            a.hint->tau = (uint32_t)(run[last] >> 32);
            a.hint->valid = run[last] != 0ull ? 1u : 0u;
        }
    } else if (a.hint && tid == 0) {
        a.hint->valid = 0u;
    }
    // scores only where the caller asked for them here (then the fleet statistics are final already)
    const float B = a.score ? a.fleet_med[pm] : 0.0f;
    const float Ds = a.score ? scale_of(a.fleet_mad[pm], B, p.floor_rel[pm], p.floor_abs[pm]) : 1.0f;
    for (int i = tid; i < K; i += blockDim.x) {
        const int r = (int)(0xFFFFFFFFu - (uint32_t)(run[i] & 0xFFFFFFFFull));
        if (a.idx) a.idx[i] = r;
        if (a.idx_keep) a.idx_keep[i] = r;
        if (a.score) {
            float dev = __fsub_rn(a.wmed[(size_t)r * a.M + pm], B);
            if (dirp < 0) dev = -dev;
            a.score[i] = (dev == 0.0f) ? 0.0f : __fdiv_rn(__fmul_rn(0.6745f, dev), Ds);
        }
    }
}


// Hinted pass (evaluations that follow one another closely: the set of slowest ranks hardly changes): every
// CTA appends the entries at or above the threshold the previous evaluation left (about three times K of
// them) to one global list; the CTA that takes the last ticket sorts the list, takes the K best and leaves the
// next threshold.  Fewer than K entries, or more than the list holds, leaves the evaluation to topk_kernel,
// which is launched right behind and returns at once otherwise.
__global__ void __launch_bounds__(kTopThreads) topk_hint_kernel(const TopkArgs a, const MetricParams p, const int nblocks) {
    __shared__ unsigned long long list[kTopChunk];
    __shared__ int is_last;
    TopkHint *h = a.hint;
    const int tid = threadIdx.x, b = blockIdx.x, lane = lane_id();
    if (!h->valid) {   // nobody writes the state in a launch that starts like this: every CTA sees the same
        if (b == 0 && tid == 0) { h->need_full = 1u; h->misses += 1u; }
        return;
    }
    const uint32_t tau = h->tau;
    const int pm = p.primary, dirp = p.dir[pm];
    const int K = a.K;
    for (int r0 = b * kTopThreads; r0 < a.R; r0 += nblocks * kTopThreads) {   // uniform trip count: the ballots below need whole warps
        const int r = r0 + tid;
        unsigned long long e = 0ull;
        bool pass = false;
        if (r < a.R) {
            float v = a.wmed[(size_t)r * a.M + pm];
            if (dirp < 0) v = -v;
            const uint32_t key = f2key(v);
            pass = key >= tau;
            e = ((unsigned long long)key << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)r);
        }
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, pass);
        if (bal) {
            uint32_t base = 0;
            if (lane == __ffs(bal) - 1) base = atomicAdd(&h->count, (uint32_t)__popc(bal));
            base = __shfl_sync(0xFFFFFFFFu, base, __ffs(bal) - 1);
            const uint32_t pos = base + __popc(bal & ((1u << lane) - 1u));
            if (pass && pos < (uint32_t)kTopChunk) a.hcand[pos] = e;
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = (atomicAdd(&h->ticket, 1u) == (unsigned)nblocks - 1u) ? 1 : 0;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int n = (int)__ldcg(&h->count);
    const bool ok = n >= K && n <= kTopChunk;
    if (ok) {
        int n2 = 2;
        while (n2 < n) n2 <<= 1;
        for (int i = tid; i < n2; i += blockDim.x) list[i] = i < n ? __ldcg(a.hcand + i) : 0ull;
        bitonic_desc(list, n2);
        for (int i = tid; i < K; i += blockDim.x) {
            const int r = (int)(0xFFFFFFFFu - (uint32_t)(list[i] & 0xFFFFFFFFull));
            if (a.idx) a.idx[i] = r;
            if (a.idx_keep) a.idx_keep[i] = r;
        }
    }
    if (tid == 0) {
        h->count = 0u;
        h->ticket = 0u;
        h->need_full = ok ? 0u : 1u;
        if (ok) {
            h->tau = (uint32_t)(list[min(n, 3 * K) - 1] >> 32);
            h->hits += 1u;
        } else {
            h->misses += 1u;
        }
    }
}

}  // namespace

int topk_blocks(int R) {
    int nb = (R + kTopChunk - 1) / kTopChunk;
    return nb < 1 ? 1 : (nb > 64 ? 64 : nb);
}

cudaError_t launch_topk(const TopkArgs &a, const MetricParams &p, cudaStream_t st) {
    if (a.K <= 0 || (!a.idx && !a.score && !a.idx_keep)) return cudaSuccess;
    const int nb = topk_blocks(a.R);
    if (a.hint && !a.score) {
        const int hb = (a.R + kTopThreads - 1) / kTopThreads;
        topk_hint_kernel<<<hb < 64 ? hb : 64, kTopThreads, 0, st>>>(a, p, hb < 64 ? hb : 64);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    topk_kernel<<<nb, kTopThreads, 0, st>>>(a, p, nb);
    return cudaGetLastError();
}

}  // namespace guard

// ---- top-k without any allocation ---------------------------------------------------------
//
// Scratch for guard_topk_static: the per-CTA candidate lists followed by the ticket word.
// It lives in the library image, so every GPU that loads the library holds these bytes
// until the process exits, and every call on a device shares them.
namespace {
constexpr int kStaticMaxBlocks = 64;   // topk_blocks() never exceeds this
constexpr size_t kStaticCandEntries = (size_t)kStaticMaxBlocks * GUARD_TOPK_STATIC_MAX_K;
constexpr size_t kStaticTicketEntries = 32;  // one 256-byte line for the ticket
static __device__ __align__(256) unsigned long long g_topk_static_scratch[kStaticCandEntries + kStaticTicketEntries];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void *g_static_ptr[kMaxDevices] = {};
}  // namespace

extern "C" int guard_topk_static(const float *d_wmed, const float *d_fleet_med, const float *d_fleet_mad, int ranks,
                                 int metrics, const guard_thresholds *th, int topk, int32_t *d_topk_idx,
                                 float *d_topk_score, void *stream) {
    using namespace guard;
    char msg[200];
    if (!d_wmed || !d_fleet_med || !d_fleet_mad || !th || !th->dir || !th->floor_rel || !th->floor_abs) {
        set_global_error("guard_topk_static: a required pointer is NULL");
        return GUARD_ERR_ARG;
    }
    if (ranks < 1 || ranks > GUARD_TOPK_STATIC_MAX_RANKS || metrics < 1 || metrics > GUARD_MAX_METRICS) {
        snprintf(msg, sizeof(msg), "guard_topk_static: need 1 <= ranks <= %d and 1 <= metrics <= %d",
                 GUARD_TOPK_STATIC_MAX_RANKS, GUARD_MAX_METRICS);
        set_global_error(msg);
        return GUARD_ERR_ARG;
    }
    if (topk < 1 || topk > GUARD_TOPK_STATIC_MAX_K || topk > ranks) {
        snprintf(msg, sizeof(msg), "guard_topk_static: topk must be in 1..min(ranks, %d); the built-in scratch holds no more",
                 GUARD_TOPK_STATIC_MAX_K);
        set_global_error(msg);
        return GUARD_ERR_ARG;
    }
    if (th->primary < 0 || th->primary >= metrics) {
        set_global_error("guard_topk_static: primary metric index out of range");
        return GUARD_ERR_ARG;
    }
    MetricParams p{};
    p.M = metrics;
    p.primary = th->primary;
    for (int m = 0; m < metrics; ++m) {
        if (th->dir[m] != 1 && th->dir[m] != -1) {
            set_global_error("guard_topk_static: dir[m] must be +1 or -1");
            return GUARD_ERR_ARG;
        }
        p.dir[m] = th->dir[m];
        p.floor_rel[m] = th->floor_rel[m];
        p.floor_abs[m] = th->floor_abs[m];
    }
    // Once per device: ask the runtime where the array lives on the current device.  In
    // host code the array's name is only a handle, never a pointer a kernel could use.
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_global_error("guard_topk_static: cudaGetDevice failed or device index out of range");
        return GUARD_ERR_CUDA;
    }
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            void *ptr = nullptr;
            e = cudaGetSymbolAddress((void **)&ptr, g_topk_static_scratch);
            if (e != cudaSuccess || !ptr) {
                snprintf(msg, sizeof(msg), "guard_topk_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
                set_global_error(msg);
                return GUARD_ERR_CUDA;
            }
            g_static_ptr[dev] = ptr;
        }
        scratch = g_static_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long *cand = (unsigned long long *)scratch;
    unsigned int *ticket = (unsigned int *)(cand + kStaticCandEntries);
    // The array keeps whatever the previous call left; only the ticket has to start at zero.
    e = cudaMemsetAsync(ticket, 0, kStaticTicketEntries * sizeof(unsigned long long), st);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof(msg), "guard_topk_static: cudaMemsetAsync: %s", cudaGetErrorString(e));
        set_global_error(msg);
        return GUARD_ERR_CUDA;
    }
    TopkArgs t{};
    t.R = ranks;
    t.M = metrics;
    t.K = topk;
    t.wmed = d_wmed;
    t.fleet_med = d_fleet_med;
    t.fleet_mad = d_fleet_mad;
    t.cand = cand;
    t.ticket = ticket;
    t.idx = d_topk_idx;
    t.score = d_topk_score;
    e = launch_topk(t, p, st);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof(msg), "guard_topk_static: launch: %s", cudaGetErrorString(e));
        set_global_error(msg);
        return GUARD_ERR_CUDA;
    }
    return GUARD_OK;
}
