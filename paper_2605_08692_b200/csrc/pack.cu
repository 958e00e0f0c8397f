// The final pack pass (Algorithm 1 lines 17-20): BF16 tables, exact selection, 4-bit codes.
//
// The tables are rounded to BF16 (RNE of the FP32 values) and sorted.  For every weight the pass
// forms w~ = fl32(w * r) (Eq. 2) and finds, with the lookup tables of lookup.cuh, the interval of
// the merged breakpoint list that holds it and the nearest entries P, Q of T0, T1 (Eq. 4).  Per
// group it sums the two activation-weighted errors (Eq. 8), picks sigma, writes the 4-bit index
// under the chosen table (Eq. 6; the index rides in the low mantissa bits of the constants the
// lookup returns) and sigma into the sign bit of the scale.
//
// Exactness.  The group errors are summed in FP32 with constants that differ from the entries by
// at most 17 * 2^-24 max|T|; groups inside the resulting error bound (see fit.cu) are re-evaluated in
// double with the exact entries, so sigma equals the double-precision decision.  The interval
// search itself is exact (rounded-down midpoints), hence so are the codes.
//
// Also reported: the Eq. 8 objective under the BF16 tables, sum_k I_k (w - w^)^2 in weight units,
// the number of groups with E0 == E1 exactly (among those re-evaluated), of weights exactly
// half-way between two different entries of their table, and of groups re-evaluated in double.
//
// Thread mapping as in the fit rounds: a block of NW warps takes items of 4 NW rows x 256 columns
// in contiguous ranges, a warp 4 rows, a lane 8 adjacent columns (one 128-bit load per row, one
// 32-bit store of 8 codes); the next item's rows are loaded while the current one is processed.
// Error sums go through one partial per block, added in block order by the last block to finish.
#include "lookup.cuh"

namespace aaac {

namespace {

// warps per block: the INT4 instance (longer shuffle reductions) gains from 16 warps at 128 registers,
// the NVFP4 instance is faster with 12 warps and its full register count
constexpr int pack_warps(int mode) { return mode == AAAC_INT4 ? 16 : 12; }
constexpr int kPackRep = 16;          // one copy of the {J_low, thr} table per lane of a half-warp: no conflicts

struct PackParams {
    const uint16_t* W;
    int64_t N, K, ldw;
    void* scales;                 // in: positive scales; out: sign bit = sigma
    const float* I;
    const float* tensor_scale;    // NVFP4
    Ctrl* ctrl;
    double* part;
    const float* T01_f32;
    uint16_t* T01_bf16;
    uint8_t* codes;
    uint8_t* sigma_bits;          // [N][K / 128] when the selection group is 16 inside a scale group of 128; else null
    int items, per_block, nrb;
};

// Number of the row's weights that lie exactly half-way between two different entries of the
// chosen table (rare; kept out of line so that the hot loop stays small).
__device__ __noinline__ int count_idx_ties(const FitTables* S, Row8 r, int sg) {
    int n = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll 1
        for (int jj = 0; jj < kNBP; ++jj)
            if (S->bp[jj] == r.x[j] && S->src[jj] == (uint8_t)sg && S->exact[jj]) { ++n; break; }
    }
    return n;
}

template <int MODE, int SEL, int NW, int REP>
__global__ void __launch_bounds__(NW * 32, 1) pack_kernel(const PackParams p) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;      // scale group
    constexpr int LPG = SEL / 8;                         // lanes per selection group
    static_assert(SEL == G || SEL == 16, "separate selection bits are laid out for groups of 16");
    constexpr int R = kRowsPerWarp;
    constexpr int kRowsPerItem = R * NW;
    constexpr int kLut1Bytes = REP * kNBins * 8;
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ FitTables S;
    __shared__ float slut[128];                      // NVFP4: s_eff per E4M3 code
    __shared__ double wsum[NW][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- BF16 tables (Algorithm 1 line 17), sorted
    float tb = 0.f;
    if (tid < 2 * kM) {
        tb = __uint_as_float(f32_to_bf16_rne(p.T01_f32[tid]) << 16);
        S.tot[tid] = (double)tb;
    }
    if (MODE == AAAC_NVFP4 && tid >= 64 && tid < 192) {
        const int c = tid - 64;
        const float sv = __fmul_rn(e4m3_value((uint32_t)c), p.tensor_scale[0]);
        slut[c] = sv;
        S.rlut[c] = c ? __frcp_rn(sv) : 0.f;
    }
    __syncthreads();
    if (tid < 2 * kM) {
        const int r = tid & 16;
        int rank = 0;
        for (int i = 0; i < kM; ++i) {
            const double ti = S.tot[r + i];
            rank += (ti < (double)tb) || (ti == (double)tb && i < (tid & 15));
        }
        S.Td[r + rank] = (double)tb;
    }
    __syncthreads();
    if (blockIdx.x == 0 && tid < 2 * kM) p.T01_bf16[tid] = (uint16_t)(__float_as_uint((float)S.Td[tid]) >> 16);
    build_tables<MODE, NW, REP>(S, dyn);

    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(dyn);
    const uint32_t lut1_lane = sm_base + (lane & (REP - 1)) * 8;
    const int c0 = (int)(sm_base + kLut1Bytes + lane * 8), c1 = c0 + kSlotBytes;
    constexpr float kMagic = 512.f + 1.5f * (float)(1 << 23) / (float)(REP * 8);
    constexpr uint32_t kBinMask = (uint32_t)(kNBins - 1) * (REP * 8);
    const float tmax283 = S.tmax283;

    double Eacc = 0.0, Eout = 0.0;
    uint32_t n_sig_tie = 0, n_idx_tie = 0, n_exact = 0;

    const int N = (int)p.N, K = (int)p.K;
    const int Gr = K / G;
    const int it0 = blockIdx.x * p.per_block;
    const int it1 = min(p.items, it0 + p.per_block);

    uint4 nv[R];
    uint32_t ns[R];           // scale bits (sign clear): E4M3 byte or BF16 pattern
    auto load_item = [&](int slab, int rb) {
        const int col0 = slab * 256 + lane * 8;
        const int row0 = rb * kRowsPerItem + warp * R;
        const uint16_t* wp = p.W + (size_t)row0 * (size_t)p.ldw + col0;
        const uint32_t g0 = (uint32_t)col0 / G;
#pragma unroll
        for (int u = 0; u < R; ++u) {
            const int row = row0 + u;
            nv[u] = make_uint4(0, 0, 0, 0);
            ns[u] = 0u;
            if (col0 < K && row < N) {
                nv[u] = __ldcs(reinterpret_cast<const uint4*>(wp + (size_t)u * (size_t)p.ldw));
                const size_t gi = (size_t)row * (size_t)Gr + g0;
                if (MODE == AAAC_NVFP4) ns[u] = reinterpret_cast<const uint8_t*>(p.scales)[gi];
                else ns[u] = reinterpret_cast<const uint16_t*>(p.scales)[gi];
            }
        }
    };

    int cur_slab = -1;
    float Iv[8];
    float isum = 0.f;
    bool col_ok = false;
#pragma unroll
    for (int j = 0; j < 8; ++j) Iv[j] = 0.f;

    int slab = it0 / p.nrb, rb = it0 - slab * p.nrb;
    int nslab = slab, nrb = rb;
    if (it0 < it1) load_item(slab, rb);
    for (int item = it0; item < it1; ++item) {
        uint4 v[R];
        uint32_t sc[R];
#pragma unroll
        for (int u = 0; u < R; ++u) { v[u] = nv[u]; sc[u] = ns[u]; }
        slab = nslab;
        rb = nrb;
        if (++nrb == p.nrb) { nrb = 0; ++nslab; }
        if (item + 1 < it1) load_item(nslab, nrb);

        const int col0 = slab * 256 + lane * 8;
        if (slab != cur_slab) {
            cur_slab = slab;
            col_ok = col0 < K;
            isum = 0.f;
            if (col_ok) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(p.I + col0));
                const float4 b = __ldg(reinterpret_cast<const float4*>(p.I + col0 + 4));
                Iv[0] = a.x; Iv[1] = a.y; Iv[2] = a.z; Iv[3] = a.w;
                Iv[4] = b.x; Iv[5] = b.y; Iv[6] = b.z; Iv[7] = b.w;
#pragma unroll
                for (int j = 0; j < 8; ++j) isum += Iv[j];
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) Iv[j] = 0.f;
            }
#pragma unroll
            for (int o = LPG / 2; o; o >>= 1) isum += __shfl_xor_sync(0xFFFFFFFFu, isum, o);
            isum *= 1.0001f;
        }
        const int row0 = rb * kRowsPerItem + warp * R;

#pragma unroll
        for (int u = 0; u < R; ++u) {
            const int row = row0 + u;
            if (row >= N) break;                            // uniform over the warp
            const uint32_t sbits = MODE == AAAC_NVFP4 ? (sc[u] & 0x7Fu) : (sc[u] & 0x7FFFu);
            float sval, rinv;
            if (MODE == AAAC_NVFP4) {
                sval = slut[sbits];
                rinv = S.rlut[sbits];
            } else {
                sval = __uint_as_float(sbits << 16);
                rinv = col_ok ? __frcp_rn(sval) : 0.f;
            }
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            float x[8];
            float2 pq[8];
            bool tcand = false;                             // some w~ equals the breakpoint of its bin
            float e0 = 0.f, e1 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                x[j] = __fmul_rn((j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]), rinv);
                const uint32_t off = (uint32_t)__float_as_int(__fmaf_rn(x[j], 64.f, kMagic)) & kBinMask;
                const uint2 e = lds_table_u2(lut1_lane + off);
                const float thr = __uint_as_float(e.y);
                tcand |= (x[j] == thr);
                pq[j] = lds_table_f2(e.x + (uint32_t)((x[j] > thr) ? c1 : c0));
                const float u0 = __fsub_rn(x[j], pq[j].x), u1 = __fsub_rn(x[j], pq[j].y);
                e0 = __fmaf_rn(__fmul_rn(Iv[j], u0), u0, e0);
                e1 = __fmaf_rn(__fmul_rn(Iv[j], u1), u1, e1);
            }
#pragma unroll
            for (int s = LPG / 2; s; s >>= 1) {
                e0 += __shfl_xor_sync(0xFFFFFFFFu, e0, s);
                e1 += __shfl_xor_sync(0xFFFFFFFFu, e1, s);
            }
            const float es = e0 + e1;
            const float tau = 0x1p-24f * __fmaf_rn(tmax283, __fsqrt_ru(__fmul_ru(isum, es)), 16.f * es);
            const bool near = !(fabsf(e1 - e0) > tau) && (col_ok || !(es == es));
            bool sg = e1 < e0;
            double emin = (double)(sg ? e1 : e0);
            if (__any_sync(0xFFFFFFFFu, near)) {
                Row8 r;
#pragma unroll
                for (int j = 0; j < 8; ++j) { r.x[j] = x[j]; r.I[j] = Iv[j]; }
                const Exact8 ex = exact_groups<LPG>(&S, r, (int)near);
                if (near) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) pq[j] = lds_table_f2((uint32_t)(c0 + ex.J[j] * kSlotBytes));
                    sg = ex.sigma != 0;
                    emin = ex.emin;
                    tcand = true;                           // poisoned slots carry no breakpoint to compare with
                    if (col_ok && (lane % LPG) == 0) { ++n_exact; n_sig_tie += ex.tie; }
                }
            }
            if (SEL != G) {
                // selection bits apart (Algorithm 1 line 20, S < g): group j of the row in bit j % 8 of
                // byte j / 8; a row's 256-column slab holds 16 groups, led by the even lanes
                uint32_t b = __ballot_sync(0xFFFFFFFFu, sg) & 0x55555555u;
                b = (b | (b >> 1)) & 0x33333333u;
                b = (b | (b >> 2)) & 0x0F0F0F0Fu;
                b = (b | (b >> 4)) & 0x00FF00FFu;
                b = (b | (b >> 8)) & 0x0000FFFFu;
                if (col_ok && (lane & 15) == 0)
                    p.sigma_bits[(size_t)row * (size_t)(K >> 7) + (uint32_t)col0 / 128u] = (uint8_t)(b >> (lane >> 1));
            }
            if (!col_ok) continue;
            if ((lane % LPG) == 0) Eacc += emin;
            // codes (Eq. 6) and the error in weight units
            uint32_t word = 0;
            float eo = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t cb = __float_as_uint(sg ? pq[j].y : pq[j].x);
                word |= (cb & kIdxMask) << (4 * j);
                const float tv = __uint_as_float((cb + 0x8000u) & 0xFFFF0000u);   // the BF16 entry itself (c is within 8 ulp of it)
                const float wf = (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]);
                const float dw = __fmaf_rn(-tv, sval, wf);
                eo = __fmaf_rn(__fmul_rn(Iv[j], dw), dw, eo);
            }
            Eout += (double)eo;
            if (tcand) {
                Row8 r;
#pragma unroll
                for (int j = 0; j < 8; ++j) { r.x[j] = x[j]; r.I[j] = 0.f; }
                n_idx_tie += count_idx_ties(&S, r, (int)sg);
            }
            *reinterpret_cast<uint32_t*>(p.codes + (((size_t)row * (size_t)K + col0) >> 1)) = word;
            if (SEL == G && (lane % LPG) == 0) {
                const size_t gi = (size_t)row * (size_t)Gr + (uint32_t)col0 / G;
                if (MODE == AAAC_NVFP4)
                    reinterpret_cast<uint8_t*>(p.scales)[gi] = (uint8_t)(sbits | (sg ? 0x80u : 0u));
                else
                    reinterpret_cast<uint16_t*>(p.scales)[gi] = (uint16_t)(sbits | (sg ? 0x8000u : 0u));
            }
        }
    }

    // ---- block partial of the two error sums; integer statistics by atomics ----
#pragma unroll
    for (int s = 16; s; s >>= 1) {
        Eacc += __shfl_xor_sync(0xFFFFFFFFu, Eacc, s);
        Eout += __shfl_xor_sync(0xFFFFFFFFu, Eout, s);
        n_sig_tie += __shfl_xor_sync(0xFFFFFFFFu, n_sig_tie, s);
        n_idx_tie += __shfl_xor_sync(0xFFFFFFFFu, n_idx_tie, s);
        n_exact += __shfl_xor_sync(0xFFFFFFFFu, n_exact, s);
    }
    if (lane == 0) {
        wsum[warp][0] = Eacc;
        wsum[warp][1] = Eout;
        if (n_sig_tie) atomicAdd(&p.ctrl->pack_stats[0], (unsigned long long)n_sig_tie);
        if (n_idx_tie) atomicAdd(&p.ctrl->pack_stats[1], (unsigned long long)n_idx_tie);
        if (n_exact) atomicAdd(&p.ctrl->pack_stats[2], (unsigned long long)n_exact);
    }
    __syncthreads();
    if (tid < 2) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < NW; ++w) s += wsum[w][tid];
        p.part[(size_t)blockIdx.x * kPartStride + tid] = s;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) S.is_last = (atomicAdd(&p.ctrl->done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!S.is_last) return;
    __threadfence();
    if (tid < 2) {
        double s = 0.0;
        for (unsigned b = 0; b < gridDim.x; ++b) s += __ldcg(p.part + (size_t)b * kPartStride + tid);
        p.ctrl->pack_err[tid] = s;
    }
    if (tid == 0) p.ctrl->done = 0;
}

__global__ void export_pack_kernel(Ctrl* ctrl, double* err_out, unsigned long long* stats) {
    if (threadIdx.x < 2 && err_out) err_out[threadIdx.x] = ctrl->pack_err[threadIdx.x];
    if (threadIdx.x < 4) {
        if (stats) stats[threadIdx.x] = ctrl->pack_stats[threadIdx.x];
        ctrl->pack_stats[threadIdx.x] = 0;
    }
}

template <int MODE, int SEL>
cudaError_t launch_pack_variant(const PackParams& p, unsigned grid, cudaStream_t st) {
    constexpr size_t smem = (size_t)kPackRep * kNBins * 8 + kJSlots * kSlotBytes;
    constexpr int kPackWarps = pack_warps(MODE);
    auto kern = pack_kernel<MODE, SEL, kPackWarps, kPackRep>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, kPackWarps * 32, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_pack(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int sel_group, const float* I,
                        const float* T01_f32, uint16_t* T01_bf16, void* scales, const float* tensor_scale,
                        uint8_t* codes, uint8_t* sigma_bits, double* err_out, unsigned long long* stats,
                        const Workspace& ws, cudaStream_t st) {
    PackParams p{};
    p.W = W; p.N = N; p.K = K; p.ldw = ldw;
    p.scales = scales; p.I = I; p.tensor_scale = tensor_scale;
    p.ctrl = ws.ctrl; p.part = ws.part; p.T01_f32 = T01_f32; p.T01_bf16 = T01_bf16; p.codes = codes;
    p.sigma_bits = sigma_bits;
    const int64_t slabs = (K + 255) / 256;
    const int kRowsPerItem = kRowsPerWarp * pack_warps(mode);
    const int64_t nrb = (N + kRowsPerItem - 1) / kRowsPerItem, items = slabs * nrb;
    if (N > 0x7FFFFFFF || K > 0x7FFFFFFF || items > 0x7FFFFFFF) return cudaErrorInvalidValue;
    int64_t grid = sm_count();
    if (grid > items) grid = items;
    if (grid > kMaxBlocks) grid = kMaxBlocks;
    const int64_t per_block = (items + grid - 1) / grid;
    grid = (items + per_block - 1) / per_block;
    p.nrb = (int)nrb; p.items = (int)items; p.per_block = (int)per_block;
    cudaError_t e;
    if (mode == AAAC_INT4 && sel_group == 16) e = launch_pack_variant<AAAC_INT4, 16>(p, (unsigned)grid, st);
    else if (mode == AAAC_INT4) e = launch_pack_variant<AAAC_INT4, 128>(p, (unsigned)grid, st);
    else e = launch_pack_variant<AAAC_NVFP4, 16>(p, (unsigned)grid, st);
    if (e != cudaSuccess) return e;
    export_pack_kernel<<<1, 32, 0, st>>>(ws.ctrl, err_out, stats);
    return cudaGetLastError();
}

}  // namespace aaac
