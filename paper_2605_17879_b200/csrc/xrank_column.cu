// Cross-rank selection, column path: one CTA of 1024 threads per (row, metric) column, the
// whole column held in registers (up to 32 values per thread, i.e. up to 32 768 ranks).
// Used when only a few rows are processed at a time -- the fleet baseline of an evaluation,
// single-step streaming ingest, the node sweep's fleet statistics -- where one CTA per row
// would leave the GPU idle and a sampled interval is not worth its set-up.
//
// The wanted order statistic is found exactly by histogram refinement on order-preserving
// keys: a 2048-bin shared-memory histogram over [min key, max key] locates the bin of the
// wanted rank, the bin becomes the new range, until a bin is a single key (three rounds for
// typical telemetry).  The MAD repeats this on |x - med|, and the exceedance bits are OR-ed
// into the (pre-zeroed) mask row, four ranks per 32-bit atomic.
#include "colreg.cuh"
#include "kernels.h"

namespace guard {

namespace {

template <int VPT, typename MaskT>
__global__ void __launch_bounds__(kColThreads) xrank_column_kernel(const XrankArgs a, const MetricParams p) {
    __shared__ ColShared sh;
    const int m = blockIdx.x, t = blockIdx.y, tid = threadIdx.x, lane = lane_id();
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const size_t col = (size_t)t * M + m;
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2);

    float x[VPT];
    uint32_t key[VPT];
    uint32_t valid = 0;
    bool bad = false;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int r = i * kColThreads + tid;
        x[i] = 0.0f;
        if (r < R) {
            x[i] = __ldg(row + (size_t)r * M + m);
            valid |= 1u << i;
            bad |= nonfinite_bits(__float_as_uint(x[i]));
        }
        key[i] = f2key(x[i]);
    }
    if (a.check_finite && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(a.status, kStatNonFinite);

    uint32_t v1, v2;
    bool ok = col_select_regs<VPT>(key, valid, k1, even, sh, v1, v2);
    const float med = median_from_keys(v1, v2, even);
    if (a.cut) {
        uint32_t c1, c2;
        ok = col_select_regs<VPT>(key, valid, (uint32_t)a.cut_rank[m], false, sh, c1, c2) && ok;
        if (tid == 0) a.cut[col] = key2f(c1);
    }
#pragma unroll
    for (int i = 0; i < VPT; ++i) key[i] = f2key(fabsf(__fsub_rn(x[i], med)));
    ok = col_select_regs<VPT>(key, valid, k1, even, sh, v1, v2) && ok;
    const float mad = median_from_keys(v1, v2, even);
    if (tid == 0) {
        if (!ok) atomicOr(a.status, kStatInternal);
        a.med[col] = med;
        a.mad[col] = mad;
        if (a.med_user) a.med_user[col] = med;
        if (a.mad_user) a.mad_user[col] = mad;
    }
    if (a.mask_base) {
        // the mask row was zeroed before the launch; the M column CTAs of a row OR their bits in
        const float rhs = __fmul_rn(p.thrp[m], scale_of(mad, med, p.floor_rel[m], p.floor_abs[m]));
        const int dir = p.dir[m];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int r = i * kColThreads + tid;
            const uint32_t e = (((valid >> i) & 1u) && exceeds(x[i], med, dir, rhs)) ? 1u : 0u;
            if (sizeof(MaskT) == 1) {
                // four adjacent ranks share a 32-bit word: combine their bits, one atomic per word
                uint32_t b = (e << m) << (8 * (tid & 3));
                b |= __shfl_xor_sync(0xFFFFFFFFu, b, 1);
                b |= __shfl_xor_sync(0xFFFFFFFFu, b, 2);
                if ((tid & 3) == 0 && b) {
                    const size_t idx = (size_t)slot * R + (size_t)r;   // r is a multiple of 4 here
                    if ((R & 3) == 0) {
                        atomicOr(reinterpret_cast<unsigned int *>(reinterpret_cast<uintptr_t>(a.mask_base) + idx), b);
                    } else {   // rows are not word aligned: fall back to one atomic per byte position
                        for (int qd = 0; qd < 4; ++qd) {
                            const uint32_t byte = (b >> (8 * qd)) & 255u;
                            if (byte) {
                                const size_t bi = idx + qd;
                                unsigned int *w = reinterpret_cast<unsigned int *>(reinterpret_cast<uintptr_t>(a.mask_base) + (bi & ~(size_t)3));
                                atomicOr(w, byte << (8 * (bi & 3)));
                            }
                        }
                    }
                }
            } else if (e) {
                atomicOr(reinterpret_cast<unsigned int *>(a.mask_base) + (size_t)slot * R + r, 1u << m);
            }
        }
    }
}

// The same with every column spread over a cluster of NC CTAs (wide fleets: one CTA per column is
// bound by instruction issue on its SM; four SMs per column share the histogram rounds through
// distributed shared memory).  CTA c of the cluster holds ranks (i * NC + c) * 1024 + tid.
template <int VPT, int NC, typename MaskT>
__global__ void __cluster_dims__(NC, 1, 1) __launch_bounds__(kColThreads)
    xrank_column_cluster_kernel(const XrankArgs a, const MetricParams p) {
    __shared__ ColShared sh;
    const int m = blockIdx.x / NC, t = blockIdx.y, tid = threadIdx.x, lane = lane_id();
    const int crank = (int)cl_rank();
    const int R = a.R, M = a.M;
    const int slot = (int)(((long long)a.first_slot + t) % a.capacity);
    const float *row = a.base + (size_t)slot * a.row_stride;
    const size_t col = (size_t)t * M + m;
    const bool even = (R & 1) == 0;
    const uint32_t k1 = (uint32_t)((R - 1) / 2);

    float x[VPT];
    uint32_t key[VPT];
    uint32_t valid = 0;
    bool bad = false;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int r = (i * NC + crank) * kColThreads + tid;
        x[i] = 0.0f;
        if (r < R) {
            x[i] = __ldg(row + (size_t)r * M + m);
            valid |= 1u << i;
            bad |= nonfinite_bits(__float_as_uint(x[i]));
        }
        key[i] = f2key(x[i]);
    }
    if (a.check_finite && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(a.status, kStatNonFinite);

    // brackets from the previous result of this call site (read before anything of this row is written)
    __shared__ HintShared hs;
    ColHintState *hst = reinterpret_cast<ColHintState *>(a.hint);
    float hc[2] = {0.0f, 0.0f}, hh[2] = {0.0f, 0.0f};
    bool hinted[2] = {false, false};
    if (hst) {
        hint_clear(hs);
        // (every CTA of the cluster reads the same state: only this cluster's own leader writes it, at the end)
        if (hst->valid[m]) {
            hc[0] = a.med[col];
            hc[1] = a.mad[col];
            // no tuned width yet: one standard error of a sample median of normal data is 1.25 x 1.4826 MAD / sqrt(R);
            // five of them for the median, three for the MAD (whose neighbourhood is 1.6 times denser)
            const float se = hc[1] * rsqrtf((float)R);
            hh[0] = hst->hw[0][m];
            hh[1] = hst->hw[1][m];
            if (hh[0] == 0.0f) hh[0] = 9.0f * se;
            if (hh[1] == 0.0f) hh[1] = 5.5f * se;
#pragma unroll
            for (int ph = 0; ph < 2; ++ph) hinted[ph] = hh[ph] >= 0.0f && hc[ph] - hh[ph] <= hc[ph] + hh[ph] && fabsf(hc[ph]) + hh[ph] < 3.0e38f;
        }
        __syncthreads();
    }
    uint32_t v1, v2, nin[2] = {0u, 0u};
    int side[2] = {0, 0};
    bool hit[2] = {false, false};
    bool ok = true;
    if (hinted[0]) hit[0] = colc_select_hinted<VPT, NC>(key, valid, k1, even, f2key(hc[0] - hh[0]), f2key(hc[0] + hh[0]), hs, 0, v1, v2, nin[0], side[0]);
    if (!hit[0]) ok = colc_select_regs<VPT, NC>(key, valid, k1, even, sh, v1, v2);
    const float med = median_from_keys(v1, v2, even);
    if (a.cut) {
        uint32_t c1, c2;
        ok = colc_select_regs<VPT, NC>(key, valid, (uint32_t)a.cut_rank[m], false, sh, c1, c2) && ok;
        if (tid == 0 && crank == 0) a.cut[col] = key2f(c1);
    }
#pragma unroll
    for (int i = 0; i < VPT; ++i) key[i] = f2key(fabsf(__fsub_rn(x[i], med)));
    if (hinted[1]) hit[1] = colc_select_hinted<VPT, NC>(key, valid, k1, even, f2key(fmaxf(hc[1] - hh[1], 0.0f)), f2key(hc[1] + hh[1]), hs, 1, v1, v2, nin[1], side[1]);
    if (!hit[1]) ok = colc_select_regs<VPT, NC>(key, valid, k1, even, sh, v1, v2) && ok;
    const float mad = median_from_keys(v1, v2, even);
    if (tid == 0 && crank == 0) {
        if (!ok) atomicOr(a.status, kStatInternal);
        a.med[col] = med;
        a.mad[col] = mad;
        if (a.med_user) a.med_user[col] = med;
        if (a.mad_user) a.mad_user[col] = mad;
        if (hst) {
            // keep about 4.5 sqrt(R) keys inside a bracket (four to five standard errors of a sample median to
            // either side for normal data); a bracket that missed is widened; one whose bins held more keys
            // than the gather lists (ties) rests for sixteen rows (negative values count up to zero)
            const float target = fminf(fmaxf(4.5f * sqrtf((float)R), 64.0f), 1500.0f);
#pragma unroll
            for (int ph = 0; ph < 2; ++ph) {
                float h = hst->hw[ph][m];
                if (hit[ph]) h = hh[ph] * fminf(fmaxf(target / (float)max(nin[ph], 1u), 0.7f), 1.5f);
                else if (hinted[ph]) h = side[ph] != 0 ? hh[ph] * 4.0f : -16.0f;
                else if (h < 0.0f) h = fminf(h + 1.0f, 0.0f);
                else h = 0.0f;
                hst->hw[ph][m] = h;
            }
            hst->valid[m] = 1;
            if (m == 0) atomicAdd(&hst->rows, 1u);
            if (hit[0] && hit[1]) atomicAdd(&hst->settled, 1u);
        }
    }
    if (a.mask_base) {
        // the mask row was zeroed before the launch; the CTAs of a row OR their bits in
        const float rhs = __fmul_rn(p.thrp[m], scale_of(mad, med, p.floor_rel[m], p.floor_abs[m]));
        const int dir = p.dir[m];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int r = (i * NC + crank) * kColThreads + tid;
            const uint32_t e = (((valid >> i) & 1u) && exceeds(x[i], med, dir, rhs)) ? 1u : 0u;
            if (sizeof(MaskT) == 1 && (R & 3) == 0) {
                // four adjacent ranks share a 32-bit word: combine their bits, one atomic per word
                uint32_t b = (e << m) << (8 * (tid & 3));
                b |= __shfl_xor_sync(0xFFFFFFFFu, b, 1);
                b |= __shfl_xor_sync(0xFFFFFFFFu, b, 2);
                if ((tid & 3) == 0 && b)
                    atomicOr(reinterpret_cast<unsigned int *>(reinterpret_cast<uintptr_t>(a.mask_base) + (size_t)slot * R + (size_t)r), b);
            } else if (e) {
                if (sizeof(MaskT) == 1) {
                    const size_t bi = (size_t)slot * R + (size_t)r;
                    unsigned int *w = reinterpret_cast<unsigned int *>(reinterpret_cast<uintptr_t>(a.mask_base) + (bi & ~(size_t)3));
                    atomicOr(w, (1u << m) << (8 * (bi & 3)));
                } else {
                    atomicOr(reinterpret_cast<unsigned int *>(a.mask_base) + (size_t)slot * R + r, 1u << m);
                }
            }
        }
    }
    if (hst) cl_sync();   // the hinted selection reads the other CTAs' lists last: none may exit before all have
}

constexpr int kColCluster = 4;

template <int VPT>
cudaError_t launch_cluster_vpt(const XrankArgs &a, const MetricParams &p, int S, cudaStream_t st) {
    const dim3 grid(a.M * kColCluster, S);
    if (a.mask_bytes == 4) xrank_column_cluster_kernel<VPT, kColCluster, uint32_t><<<grid, kColThreads, 0, st>>>(a, p);
    else xrank_column_cluster_kernel<VPT, kColCluster, uint8_t><<<grid, kColThreads, 0, st>>>(a, p);
    return cudaGetLastError();
}

template <int VPT>
cudaError_t launch_vpt(const XrankArgs &a, const MetricParams &p, int S, cudaStream_t st) {
    const dim3 grid(a.M, S);
    if (a.mask_bytes == 4) xrank_column_kernel<VPT, uint32_t><<<grid, kColThreads, 0, st>>>(a, p);
    else xrank_column_kernel<VPT, uint8_t><<<grid, kColThreads, 0, st>>>(a, p);
    return cudaGetLastError();
}

}  // namespace

bool xrank_column_supported(int R) { return R >= 1024 && R <= 32 * kColThreads; }

// Zeroes the exceedance rows of the S steps (at most two memsets when the span wraps), then
// runs one CTA per column (or one cluster per column: the widest columns, and single rows whose call
// site keeps a bracket from its previous result).
cudaError_t launch_xrank_column(const XrankArgs &a, const MetricParams &p, int S, cudaStream_t st) {
    if (S <= 0) return cudaSuccess;
    if (a.mask_base) {
        const size_t rowb = (size_t)a.R * a.mask_bytes;
        const int first = a.first_slot % a.capacity;
        const int n1 = (first + S <= a.capacity) ? S : (a.capacity - first);
        cudaError_t e = cudaMemsetAsync((char *)a.mask_base + (size_t)first * rowb, 0, (size_t)n1 * rowb, st);
        if (e == cudaSuccess && n1 < S) e = cudaMemsetAsync(a.mask_base, 0, (size_t)(S - n1) * rowb, st);
        if (e != cudaSuccess) return e;
    }
    const int vpt = (a.R + kColThreads - 1) / kColThreads;
    // the widest columns (more than 16 keys per thread of a single CTA) take a cluster of four CTAs each:
    // measured 45 -> 35 us per launch at 32 768 ranks; at 16 384 ranks the cluster barriers cost more than
    // the shared work saves (node sweep 0.13 -> 0.18 ms), so narrower columns stay with one CTA
    if (vpt > 16) return launch_cluster_vpt<8>(a, p, S, st);
    // a single row with a bracket from the previous result of its call site: the hinted selection of the cluster
    // kernel needs two cluster barriers per statistic, which pays from 8 192 ranks on
    if (a.hint && S == 1 && a.R >= 8192) {
        const int cv = (a.R + kColCluster * kColThreads - 1) / (kColCluster * kColThreads);
        return cv <= 2 ? launch_cluster_vpt<2>(a, p, S, st) : launch_cluster_vpt<4>(a, p, S, st);
    }
    if (vpt <= 4) return launch_vpt<4>(a, p, S, st);
    if (vpt <= 8) return launch_vpt<8>(a, p, S, st);
    if (vpt <= 16) return launch_vpt<16>(a, p, S, st);
    return launch_vpt<32>(a, p, S, st);
}

}  // namespace guard
