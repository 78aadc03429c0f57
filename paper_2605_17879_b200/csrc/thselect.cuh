// One thread per series: counting / keeping cell operation and the selection among the kept keys of a
// thread's shared-memory column (the same instruction stream in every lane of a warp).
#pragma once
#include "common.cuh"

namespace guard {

// cnt += (x < lo); if (lo <= x <= hi) { if (addr < lim) shared[addr] = x; addr += 4; }
__device__ __forceinline__ void th_cell(const float x, const float lo, const float hi, const uint32_t lim, uint32_t &cnt,
                                        uint32_t &addr) {
    asm volatile(
        "{\n\t.reg .pred p, q, r;\n\t"
        "setp.lt.f32 p, %2, %3;\n\t"
        "setp.le.and.f32 q, %2, %4, !p;\n\t"
        "setp.lt.and.u32 r, %1, %5, q;\n\t"
        "@p add.u32 %0, %0, 1;\n\t"
        "@r st.shared.f32 [%1], %2;\n\t"
        "@q add.u32 %1, %1, 4;\n\t}"
        : "+r"(cnt), "+r"(addr)
        : "f"(x), "f"(lo), "f"(hi), "r"(lim)
        : "memory");
}
__device__ __forceinline__ uint4 th_lds4(const uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void th_sts4(const uint32_t addr, const uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// The keys of ranks t - 1 (vb) and t (vu) among the nk kept values (raw float bits, all inside [klo, khi] as keys) of
// the column at shared-memory address kbase (SLOTS words, 16-byte aligned).  Lanes with ok == false take part
// without a result; ok turns false if the selection does not converge.  All 32 lanes of the warp call this together.
template <int SLOTS, int MAXPASS>
__device__ __forceinline__ void th_select_pair(const uint32_t kbase, const int nk, bool &ok, const int t, const uint32_t klo,
                                               const uint32_t khi, uint32_t &vb, uint32_t &vu) {
    const int nkmax = (int)__reduce_max_sync(0xFFFFFFFFu, ok ? (uint32_t)nk : 0u);
    if (nkmax > 0) {
        const int nkr = (nkmax + 3) & ~3;   // <= SLOTS (a multiple of 4)
        for (int j = 0; j < nkr; j += 4) {  // raw bits -> keys; slots without a key compare above everything
            uint4 v = th_lds4(kbase + 4u * j);
            v.x = (ok && j + 0 < nk) ? key_of_bits(v.x) : 0xFFFFFFFFu;
            v.y = (ok && j + 1 < nk) ? key_of_bits(v.y) : 0xFFFFFFFFu;
            v.z = (ok && j + 2 < nk) ? key_of_bits(v.z) : 0xFFFFFFFFu;
            v.w = (ok && j + 3 < nk) ? key_of_bits(v.w) : 0xFFFFFFFFu;
            th_sts4(kbase + 4u * j, v);
        }
        // The pivot moves inside a key bracket (pl, ph) with below(pl) = al <= t - 2 and
        // below(ph) = ah >= t + 2.
        uint32_t pl = klo, ph = khi + 1u, pv = klo;
        int al = 0, ah = nk, bsave = 0;
        int done = 0;                 // 1: pv has bsave in {t - 1, t, t + 1} keys below it, 2: both ranks equal pl
        if (!ok || t <= 1) { done = 1; pv = klo; bsave = 0; }
        else if (t >= nk - 1) { done = 1; pv = khi + 1u; bsave = nk; }
        for (int pass = 0; pass < MAXPASS; ++pass) {
            if (__all_sync(0xFFFFFFFFu, done != 0)) break;
            if (!done) {
                if (ph - pl < 2u) {
                    done = 2;
                } else if (pass % 3 == 2) {
                    pv = pl + ((ph - pl) >> 1);
                } else {   // aim between the ends in proportion to the missing count
                    const float fr = (float)(t - al) / (float)(ah - al);
                    pv = pl + (uint32_t)((float)(ph - pl) * fr);
                    pv = pv <= pl ? pl + 1u : (pv >= ph ? ph - 1u : pv);
                }
            }
            // the loads of a third of the column are issued before their compares
            int below = 0;
#pragma unroll
            for (int j0 = 0; j0 < SLOTS / 4; j0 += 5) {
                uint4 kv4[5];
#pragma unroll
                for (int j = 0; j < 5; ++j)
                    if (4 * (j0 + j) < nkr) kv4[j] = th_lds4(kbase + 16u * (j0 + j));
#pragma unroll
                for (int j = 0; j < 5; ++j)
                    if (4 * (j0 + j) < nkr) below += (kv4[j].x < pv) + (kv4[j].y < pv) + (kv4[j].z < pv) + (kv4[j].w < pv);
            }
            if (!done) {
                if (below >= t - 1 && below <= t + 1) { done = 1; bsave = below; }
                else if (below < t) { pl = pv; al = below; }
                else { ph = pv; ah = below; }
            }
        }
        if (ok && !done) {
            if (ph - pl < 2u) done = 2; else ok = false;
        }
        // the two largest keys below the pivot (b1 >= b2), the two smallest keys not below it (u1 <= u2)
        uint32_t b1 = 0u, b2 = 0u, u1 = 0xFFFFFFFFu, u2 = 0xFFFFFFFFu;
        for (int j = 0; j < nkr; j += 4) {
            const uint4 v4 = th_lds4(kbase + 4u * j);
            const uint32_t v[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool lt = v[u] < pv;
                const uint32_t lo_v = lt ? v[u] : 0u, hi_v = lt ? 0xFFFFFFFFu : v[u];   // neutral on the other side
                b2 = max(b2, min(b1, lo_v));
                b1 = max(b1, lo_v);
                u2 = min(u2, max(u1, hi_v));
                u1 = min(u1, hi_v);
            }
        }
        vb = b1; vu = u1;                                // bsave == t
        if (bsave == t + 1) { vb = b2; vu = b1; }
        if (bsave == t - 1) { vb = u1; vu = u2; }
        if (done == 2) { vb = pl; vu = pl; }
    }
}

}  // namespace guard
