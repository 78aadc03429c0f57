// Declarations shared by the split cross-rank path (xrank_split.cu: sample, sweeps, selections, finish)
// and the tile kernels that replace its sweeps on the large-block path (xrank_tile.cu).
#pragma once
#include "xrank_common.cuh"
#include "kernels.h"

namespace guard {

constexpr int kSpThreads = 256;     // sweep CTA
constexpr int kSpU = 4;             // ranks per thread and sweep batch
constexpr int kSpSlice = 4096;      // ranks per sweep CTA
constexpr int kSpSlack = 128;       // words behind each shared-memory list that absorb the stores of a full list
constexpr int kSpAmb = 1024;        // deferred exceedance decisions per step
constexpr int kSpSample = 4096;     // target number of sampled ranks per column
constexpr int kSpSBins = 2048;      // sample histogram bins (16-bit counters, two per word)
constexpr int kSpBins = 1024;       // selection histogram bins
constexpr int kSpSelThreads = 128;  // sample / select CTA
constexpr int kSpJmax = 20;         // kept elements per thread the register selection can hold
constexpr int kSpSegs = 4;          // sweep CTAs per step the selection can gather from
constexpr int kSpMaxM = 8;
constexpr float kFltMax = 3.402823466e+38f;

struct SpGeom {
    int chunks;     // sweep CTAs per step
    int slice;      // ranks per sweep CTA (a multiple of 16)
    int cap;        // kept elements per metric and sweep CTA (its shared-memory list and its segment in global scratch)
    int stride;     // one run of four consecutive ranks is sampled out of every 4 * stride
    int s;          // number of sampled ranks
    int delta;      // half-width of the median interval in sample ranks
    int delta_q;    // half-width of the quartile intervals in sample ranks
};

// Per-column record in global scratch.
struct SpCol {
    float lo, hi, dlo, dhi;   // intervals of the median and of the MAD
    float med, rlo, rhi, rhs; // median; range of the exceedance threshold over [dlo, dhi]; exact threshold
    uint32_t cnt;             // elements below the current interval
    uint32_t pad[3];
};

struct SpScratch {
    SpCol *col;       // [S][M]
    uint32_t *fail;   // [S] the step goes to the direct path
    uint32_t *namb;   // [S] deferred exceedance decisions
    uint32_t *amb;    // [S][kSpAmb] (rank << 5 | metric)
    uint32_t *nseg;   // [S][M][chunks] kept elements of each sweep CTA
    uint32_t *list;   // [S][M][chunks][cap] kept elements (raw bits), one segment per sweep CTA
    // tile path (NULL / 0 when the block takes the chunked sweeps)
    unsigned long long *cnt64;   // [2][S][M / 4] packed counts below the interval
    unsigned long long *nk64;    // [2][S][M / 4] packed numbers of kept elements
    uint32_t *clist;             // [S][M][kTileCap] kept elements of a column, contiguous
    float *blo, *bhi, *bdlo, *bdhi;   // [S][M] the columns' intervals again, metric-contiguous (128-bit loads)
    float *bmed, *brlo;               // [S][M] medians and lower ends of the threshold ranges, likewise
    int tile;
};

// ---- tile path: the sweeps as one kernel per rank tile over all steps of the block ---------------
// Below-interval counts and kept-element counts of a (step, four metrics) quad are packed into one
// 64-bit word, 16 bits per metric (fleets of at most 65 535 ranks), so that a tile adds its share of
// four columns with one atomic; index [mode][step][quad], mode 0 = median pass, 1 = MAD pass.
constexpr int kTileCap = 2560;        // kept elements per column (the register selection's capacity)
constexpr int kTileMinSteps = 48;     // shorter blocks stay with the chunked sweeps

// Window medians fused into the median pass of the tile kernel (the block is the evaluation's window).
struct TileWindow {
    int enabled;          // 0: cross-rank work only
    int n;                // window length: the last n steps of the block
    float *wmed;          // [series] out
    float *spread;        // [series] state: half-width of the search interval
    float *centre;        // [series] state: centre of the search interval
    int target;           // keys the interval is tuned to catch (0: default)
    float smooth;         // weight of the newest median in the centre (0: default)
    uint32_t *fb_count;   // [6] diagnostic counters or NULL
};

bool xrank_tile_supported(int R, int M, int S);
// mode 0: counts / keeps against [lo, hi] (and the window medians if win.enabled);
// mode 1: the same for |x - med| against [dlo, dhi], plus exceedance bits and the finite check.
cudaError_t launch_xtile_sweep(int mode, const XrankArgs &a, const MetricParams &p, const SpScratch &sc, int S,
                               const TileWindow &win, cudaStream_t st);

}  // namespace guard
