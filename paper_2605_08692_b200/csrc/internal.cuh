// Shared device helpers and launcher declarations of the AAAC sm_100a library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/aaac.h"

namespace aaac {

constexpr int kM = 16;            // entries per table
constexpr int kNBP = 30;          // merged breakpoints: 15 midpoints of T0 + 15 of T1
constexpr int kNJ = 31;           // merged intervals
constexpr int kPartStride = 128;  // doubles per block partial (pack: [2][31] S, Wt, E; fit: [32] S, [32] Wt, E)
constexpr int kMaxBlocks = 2048;  // upper bound on fit-kernel grid size
constexpr int kQBins = 16384;     // first-level histogram bins of the quantile selection
constexpr int kQReq = 64;         // order statistics requested (2 per table entry)
constexpr int kActMaxSplits = 32;   // row strips of the activation statistics (the second kernel adds them one after the other)

// shape of the fit-round kernel: warps per block, copies of the {J_low, thr} table
#ifndef AAAC_FIT_WARPS
#define AAAC_FIT_WARPS 16
#endif
#ifndef AAAC_FIT_REP
#define AAAC_FIT_REP 16           // one copy per lane of a half-warp: an 8-byte lookup has no bank conflicts
#endif
#ifndef AAAC_FIT_BINS
#define AAAC_FIT_BINS 512         // uniform bins of the {J_low, thr} table on (-8, 8): width 1/32
#endif

// ---- control block at the start of the workspace (device memory) ----
struct Ctrl {
    double T[2 * kM];               // current tables (double between rounds)
    float s_t;                      // NVFP4 tensor scale
    uint32_t absmax_bits;           // layer max |w| as float bits (atomicMax on non-negative floats)
    uint32_t done;                  // blocks that have written their partial this round
    uint32_t nonfinite;             // set if a non-finite weight was seen
    uint32_t bar;                   // (unused)
    uint32_t abort;                 // set when a block's wait for the totals of a pass ran out
    // quantile selection
    unsigned long long rank[kQReq]; // requested 0-based ranks (host-written via kernel args)
    double frac[2 * kM];            // interpolation fraction per table entry
    float rank_val[kQReq];          // selected order statistics
    uint32_t req_slot[kQReq];       // slot of each request
    unsigned long long req_local[kQReq];   // rank inside the slot's list
    uint32_t nslots;
    unsigned long long slot_off[kQReq + 1];
    uint32_t slot_fill[kQReq];
    uint32_t slot_over[kQReq];      // the slot's candidates did not fit the list: only their smallest and largest key are kept
    uint32_t slot_kmin[kQReq], slot_kmax[kQReq];
    uint32_t scratch_short;         // an order statistic could not be found within the scratch given
    // pack results
    double pack_err[2];
    unsigned long long pack_stats[4];
};

struct Workspace {
    Ctrl* ctrl;
    double* part;            // [kMaxBlocks][kPartStride]: the pack pass's block partials; the fit rounds' sum buffers
    float* rinv;             // [N*K/g]  INT4 reciprocal scales (one element in NVFP4 mode)
    float* I;                // [K] importance computed from X
    double* act_part;        // [kActMaxSplits][K]
    uint32_t* qhist;         // [kQBins]
    uint8_t* qslot_of_bin;   // [kQBins]
    uint32_t* qlist;         // [qcap] candidates of the quantile selection; afterwards the fit's selection bits [N][ceil(K/256)]
    size_t qcap;             // entries of qlist
    size_t bytes;
};

// ---- formats ----
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t f32_to_bf16_rne(float f) {
    uint32_t u = __float_as_uint(f);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return u >> 16;
}

// E4M3 (no infinities, 0x7F = NaN): value of a code with the sign bit already removed
__device__ __forceinline__ float e4m3_value(uint32_t c) {
    uint32_t e = (c >> 3) & 15u, m = c & 7u;
    return e ? __uint_as_float(((e + 120u) << 23) | (m << 20)) : (float)m * 0.001953125f;
}

// nearest-even E4M3 code of a finite x >= 0, saturating at 448 (0x7E)
__device__ __forceinline__ uint32_t e4m3_encode(float x) {
    if (!(x < 448.f)) return 0x7Eu;
    if (x < 0.015625f) return (uint32_t)__float2int_rn(x * 512.f);   // subnormal step 2^-9; 8 -> 2^-6
    uint32_t u = __float_as_uint(x);
    u += 0x7FFFFu + ((u >> 20) & 1u);
    u = (u >> 20) - 960u;                                            // rebias 127 -> 7
    return u > 0x7Eu ? 0x7Eu : u;
}

// bin = floor(1024 x + 8192): one multiply-add rounded down onto 1.5 * 2^23 (where floats are
// spaced by 1) leaves the integer in the low mantissa bits; the mask keeps any input inside the
// table (|w~| < 8 by the scale rules, so for finite weights it changes nothing)
__device__ __forceinline__ int qbin(float x) {
    return (int)(__float_as_uint(__fmaf_rd(x, 1024.f, 8192.f + 12582912.f)) & (uint32_t)(kQBins - 1));
}

// Walks the items first, first + stride, first + 2 stride, ... of an N x slabs grid (row-major)
// without a division per step; row runs past N when the walk is over.
struct SlabWalk {
    int row, slab, drow, dslab, slabs;
    __device__ SlabWalk(int64_t first, int64_t stride, int64_t slabs_)
        : row((int)(first / slabs_)), slab((int)(first % slabs_)), drow((int)(stride / slabs_)),
          dslab((int)(stride % slabs_)), slabs((int)slabs_) {}
    __device__ void next() {
        row += drow;
        slab += dslab;
        if (slab >= slabs) { slab -= slabs; ++row; }
    }
};

// largest float <= d
__device__ __forceinline__ float f32_round_down(double d) { return __double2float_rd(d); }

// ---- launchers (each enqueues on `st` and returns the launch status) ----
cudaError_t launch_act_stats(const uint16_t* X, int64_t T, int64_t K, int64_t ldx, float* I, int accumulate,
                             uint32_t* dev_status, const Workspace& ws, cudaStream_t st);
// with_hist: the scales pass also counts the 16384-bin histogram of the normalised weights (the quantile
// start's first pass over W) into ws.qhist; launch_init is then told so
cudaError_t launch_scales(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, void* scales,
                          float* tensor_scale, uint32_t* dev_status, const Workspace& ws, cudaStream_t st, bool with_hist = false);
cudaError_t launch_init(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int init,
                        const void* scales, const float* T01_user, uint32_t* dev_status, const Workspace& ws, cudaStream_t st,
                        bool hist_done = false);
int act_splits_max(int64_t K);    // most row strips launch_act_stats uses for K input channels (sizes its partials)
cudaError_t launch_fit_rounds(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int sel_group, const void* scales,
                              const float* I, int n_outer, int n_inner, double* err_trace, float* T01_out, uint32_t* dev_status,
                              const Workspace& ws, cudaStream_t st);
// the same for several layers of one mode in a single launch (n_inner = 1; otherwise layer by layer)
struct FitLayerArgs {
    const uint16_t* W;
    int64_t N, K, ldw;
    const void* scales;
    const float* I;
    double* err_trace;
    float* T01_out;          // where the fitted tables go as FP32 (written by the last launch), or null
    Workspace ws;
};
cudaError_t launch_fit_rounds_batch(const FitLayerArgs* layers, int n, int mode, int sel_group, int n_outer, int n_inner,
                                    uint32_t* dev_status, cudaStream_t st);
cudaError_t launch_export_tables(float* T01, const Workspace& ws, cudaStream_t st);
// sigma_bits: null when the selection group is the scale group (sigma in the scale's sign bit)
cudaError_t launch_pack(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int sel_group, const float* I,
                        const float* T01_f32, uint16_t* T01_bf16, void* scales, const float* tensor_scale,
                        uint8_t* codes, uint8_t* sigma_bits, double* err_out, unsigned long long* stats,
                        const Workspace& ws, cudaStream_t st);
cudaError_t launch_dequant(const uint8_t* codes, const void* scales, const uint8_t* sigma_bits,
                           const float* tensor_scale, const uint16_t* Tb, int64_t N, int64_t K, int mode,
                           uint16_t* What, int64_t ldo, cudaStream_t st);

cudaError_t launch_prescale(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, const float* a, uint16_t* Wout,
                            int64_t ldo, const float* I, float* Iout, uint32_t* dev_status, cudaStream_t st);

int sm_count();
void note_launch(int n = 1);      // counts kernel launches (aaac_launch_count)
void set_fit_wait(int extra_arrivals, unsigned spin_limit);   // knobs of the fit rounds' bounded wait (aaac_debug_fit_wait)

}  // namespace aaac
