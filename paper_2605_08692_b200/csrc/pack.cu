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
// Also reported: the Eq. 8 objective under the BF16 tables, sum_k I_k (w - w^)^2 in weight units
// (per group s^2 times the group's Eq. 8 error: w - w^ = s (w~ - T) up to the 2^-23 rounding of w~),
// the number of groups with E0 == E1 exactly (among those re-evaluated), of weights exactly
// half-way between two different entries of their table, and of groups re-evaluated in double.
//
// Thread mapping.  The pass keeps no bins, so its lookup tables (512 bins) leave room for two
// blocks of 8 warps per SM, and memory and table latency are hidden by the number of warps rather
// than by a hand-built pipeline: a warp walks down the rows of one 256-column slab (so its eight
// importances stay in registers), two rows per trip in registers of their own -- while one is worked
// on, the other's load is in flight and nothing is copied -- with 32-bit element offsets advanced by
// the row stride and no branch around the loads; a lane takes 8 adjacent columns (one 128-bit load per row, one 32-bit store of 8 codes); the two errors travel
// as one packed FP32 pair.
// Error sums go through one partial per block, added in block order by the last block to finish.
#include "lookup.cuh"

namespace aaac {

namespace {

// warps per block
#ifndef AAAC_PACK_WARPS
#define AAAC_PACK_WARPS 8
#endif
constexpr int pack_warps(int) { return AAAC_PACK_WARPS; }
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
    double* err_out;              // [2] or null
    unsigned long long* stats;    // [4] or null
};

// The rare path of a row, out of line so that the hot loop holds a single call: for the lanes that
// ask (flags != 0) the interval of every weight is found by binary search of the breakpoint list;
// the groups flagged kNear are decided in double (Eq. 8 as a plain double-precision loop states
// it, the lanes of a group combined by a shuffle tree); and for every asking lane the weights that
// lie exactly half-way between two different entries of the chosen table are counted (x equals a
// breakpoint that is an exact midpoint of that table).  Every lane of the warp calls.
constexpr int kNear = 1, kTieCand = 2, kFastSigma = 4;
struct Rare8 { int J[8]; double emin; int sigma; int tie; int nties; };

template <int LPG>
__device__ __noinline__ Rare8 rare_groups(const FitTables* S, Row8 r, int flags) {
    Rare8 out;
    const bool need = (flags & (kNear | kTieCand)) != 0, near = (flags & kNear) != 0;
    double e0 = 0.0, e1 = 0.0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        int J = 0;
        if (need) {
            if (r.hint[j] < (uint32_t)kNJ) {
                J = (int)r.hint[j];
            } else {
#pragma unroll
                for (int step = 16; step; step >>= 1)      // number of breakpoints below x (sorted list)
                    if (J + step <= kNBP && S->bp[J + step - 1] < r.x[j]) J += step;
            }
            if (near) {
                const double2 pq = S->PQ[J];
                const double xd = (double)r.x[j], id = (double)r.I[j];
                const double d0 = __dsub_rn(xd, pq.x), d1 = __dsub_rn(xd, pq.y);
                e0 = __dadd_rn(e0, __dmul_rn(id, __dmul_rn(d0, d0)));
                e1 = __dadd_rn(e1, __dmul_rn(id, __dmul_rn(d1, d1)));
            }
        }
        out.J[j] = J;
    }
#pragma unroll
    for (int s = LPG / 2; s; s >>= 1) {
        e0 = __dadd_rn(e0, __shfl_xor_sync(0xFFFFFFFFu, e0, s));
        e1 = __dadd_rn(e1, __shfl_xor_sync(0xFFFFFFFFu, e1, s));
    }
    out.sigma = near ? (int)(e1 < e0) : ((flags & kFastSigma) != 0);
    out.tie = near && e0 == e1;
    out.emin = out.sigma ? e1 : e0;
    int n = 0;
    if (need) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            for (int jj = out.J[j]; jj < kNBP && S->bp[jj] == r.x[j]; ++jj)     // the breakpoints equal to x, if any
                if (S->src[jj] == (uint8_t)out.sigma && S->exact[jj]) { ++n; break; }
    }
    out.nties = n;
    return out;
}

constexpr int kPackBins = 512;        // uniform bins of the per-bin table on (-8, 8): width 1/32
constexpr int kPackBlocksPerSM = 2;

template <int MODE, int SEL, int NW, int REP>
__global__ void __launch_bounds__(NW * 32, kPackBlocksPerSM) pack_kernel(const PackParams p) {
    constexpr int NB = kPackBins;
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;      // scale group
    constexpr int LPG = SEL / 8;                         // lanes per selection group
    static_assert(SEL == G || SEL == 16, "separate selection bits are laid out for groups of 16");
    constexpr int kLut1Bytes = REP * NB * 8;
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
    build_tables<MODE, NW, REP, NB>(S, dyn);

    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(dyn);
    const uint32_t lut1_copy = (lane & (REP - 1)) * 8;             // this lane's copy of a bin's entry
    const uint32_t lut2_addr = sm_base + kLut1Bytes;                // the {P, Q} table
    constexpr float kBinsPerUnit = (float)(NB / 16);
    constexpr float kMagic = (float)(NB / 2) + 1.5f * (float)(1 << 23) / (float)(REP * 8);
    constexpr uint32_t kBinMask = (uint32_t)(NB - 1) * (REP * 8);
    // near-tie bound (see fit.cu): |E0 - E1| <= g1 (E0 + E1) + g2 sum I sends the group to the double path
    const float g1 = 0x1p-24f * __fmaf_ru(S.tmax283, 4.f, 16.f), g2 = 0x1p-24f * __fmul_ru(S.tmax283, 0.0625f);

    double Eacc = 0.0, Eout = 0.0;
    uint32_t n_sig_tie = 0, n_idx_tie = 0, n_exact = 0;

    const int N = (int)p.N, K = (int)p.K;
    const int Gr = K / G;
    const int slabs = (K + 255) >> 8;
    // Warp w of the grid takes slab w mod slabs and, of the warps that share that slab, every
    // (warps per slab)-th row; with fewer warps than slabs a warp takes several slabs in turn.
    const int gw = blockIdx.x * NW + warp, nw_total = gridDim.x * NW;

    for (int slab = gw % slabs; slab < slabs; slab += nw_total) {
        // the rows of the slab are dealt to the warps that share it (those with the same index mod
        // slabs): warp number `my` of `per_slab` takes rows my, my + per_slab, ...
        const int per_slab = nw_total >= slabs ? (nw_total - (gw % slabs) + slabs - 1) / slabs : 1;
        const int my = nw_total >= slabs ? gw / slabs : 0;
        const int col0 = slab * 256 + lane * 8;
        const bool col_ok = col0 < K;
        uint64_t II[8];                       // {I, I} of the lane's eight columns
        float isum = 0.f;                     // g2 * sum of I over the lane's selection group (rounded up a little)
        {
            float Iv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) Iv[j] = 0.f;
            if (col_ok) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(p.I + col0));
                const float4 b = __ldg(reinterpret_cast<const float4*>(p.I + col0 + 4));
                Iv[0] = a.x; Iv[1] = a.y; Iv[2] = a.z; Iv[3] = a.w;
                Iv[4] = b.x; Iv[5] = b.y; Iv[6] = b.z; Iv[7] = b.w;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) { isum += Iv[j]; II[j] = pack2(Iv[j], Iv[j]); }
#pragma unroll
            for (int o = LPG / 2; o; o >>= 1) isum += __shfl_xor_sync(0xFFFFFFFFu, isum, o);
            isum = __fmul_ru(isum * 1.0001f, g2);
        }
        // Element offsets of this lane's piece of the current row, advanced by the row stride (a layer of
        // 2^32 elements or more is refused by the entry point); lanes past K read the slab's last valid
        // columns instead (their importances are zero and they write nothing).
        const unsigned col_ld = (unsigned)min(col0, K - 8);
        const unsigned step_w = (unsigned)per_slab * (unsigned)p.ldw, step_g = (unsigned)per_slab * (unsigned)Gr;
        const unsigned step_c = (unsigned)per_slab * (unsigned)(K >> 1);
        const uint16_t* const Wp = p.W;
        auto load = [&](unsigned wo, unsigned go, uint4& v, uint32_t& sc) {
            v = __ldcs(reinterpret_cast<const uint4*>(Wp + wo));
            if (MODE == AAAC_NVFP4) sc = reinterpret_cast<const uint8_t*>(p.scales)[go];
            else sc = reinterpret_cast<const uint16_t*>(p.scales)[go];
        };
        float ef = 0.f, eof = 0.f;            // the two error sums of up to 16 rows (one conversion to double per 16 rows)
        int nrow = 0;
        // one row: v and scv were loaded before; (wo, go) are the row's offsets, co the byte offset of its codes
        auto do_row = [&](const uint4& v, uint32_t scv, int row, unsigned go, unsigned co) {
            const uint32_t sbits = MODE == AAAC_NVFP4 ? (scv & 0x7Fu) : (scv & 0x7FFFu);
            float sval, rinv;
            if (MODE == AAAC_NVFP4) {
                sval = slut[sbits];
                rinv = S.rlut[sbits];
            } else {
                sval = __uint_as_float(sbits << 16);
                rinv = __frcp_rn(sval);
            }
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            float x[8];
            uint64_t pq[8];
            bool tcand = false;                             // some w~ equals the breakpoint of its bin
            uint64_t e01 = 0ull;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                x[j] = __fmul_rn((j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]), rinv);
                const uint32_t off = ((uint32_t)__float_as_int(__fmaf_rn(x[j], kBinsPerUnit, kMagic)) & kBinMask) | lut1_copy;
                const uint2 e = lds_table_u2(sm_base + off);
                tcand |= (x[j] == __uint_as_float(e.y));
                pq[j] = lds_table_b64(above_addr(e.x, x[j], e.y));
                const uint64_t u01 = diff2(x[j], pq[j]);
                e01 = fma2(mul2(II[j], u01), u01, e01);
            }
            float e0 = lo2(e01), e1 = hi2(e01);
#pragma unroll
            for (int s2 = LPG / 2; s2; s2 >>= 1) {
                e0 += __shfl_xor_sync(0xFFFFFFFFu, e0, s2);
                e1 += __shfl_xor_sync(0xFFFFFFFFu, e1, s2);
            }
            const float es = e0 + e1;
            const float tau = __fmaf_ru(es, g1, isum);
            const bool near = !(fabsf(e1 - e0) > tau) && (col_ok || !(es == es));
            bool sg = e1 < e0;
            float emin = sg ? e1 : e0;
            if (__any_sync(0xFFFFFFFFu, near || tcand)) {
                // near-ties, poisoned slots and weights that sit on a breakpoint (rare, out of line)
                Row8 r;
#pragma unroll
                for (int j = 0; j < 8; ++j) { r.x[j] = x[j]; r.I[j] = lo2(II[j]); r.hint[j] = interval_hint(S, pq[j]); }
                const Rare8 ex = rare_groups<LPG>(&S, r, (near ? kNear : 0) | (tcand ? kTieCand : 0) | (sg ? kFastSigma : 0));
                if (near) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) pq[j] = lds_table_b64(pq_entry_addr(lut2_addr, ex.J[j], lane));
                    sg = ex.sigma != 0;
                    emin = (float)ex.emin;
                    if (col_ok && (lane % LPG) == 0) { ++n_exact; n_sig_tie += ex.tie; }
                }
                if (col_ok) n_idx_tie += ex.nties;
            }
            if (SEL != G) {
                // selection bits apart (Algorithm 1 line 20, S < g): group j of the row in bit j % 8 of
                // byte j / 8; a row's 256-column slab holds 16 groups, led by the even lanes
                uint32_t bb = __ballot_sync(0xFFFFFFFFu, sg) & 0x55555555u;
                bb = (bb | (bb >> 1)) & 0x33333333u;
                bb = (bb | (bb >> 2)) & 0x0F0F0F0Fu;
                bb = (bb | (bb >> 4)) & 0x00FF00FFu;
                bb = (bb | (bb >> 8)) & 0x0000FFFFu;
                if (col_ok && (lane & 15) == 0)
                    p.sigma_bits[(size_t)row * (size_t)(K >> 7) + (uint32_t)col0 / 128u] = (uint8_t)(bb >> (lane >> 1));
            }
            if (!col_ok) return;
            if ((lane % LPG) == 0) {
                // both error sums from the group's smaller error: sum I (w - w^)^2 = s^2 sum I (w~ - T)^2
                ef += emin;
                eof = __fmaf_rn(emin, __fmul_rn(sval, sval), eof);
            }
            // codes (Eq. 6): the entry index rides in the low mantissa bits of the chosen constant
            uint32_t word = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float cP, cQ;
                unpack2(pq[j], cP, cQ);
                word |= (__float_as_uint(sg ? cQ : cP) & kIdxMask) << (4 * j);
            }
            *reinterpret_cast<uint32_t*>(p.codes + co) = word;
            if (SEL == G && (lane % LPG) == 0) {
                if (MODE == AAAC_NVFP4)
                    reinterpret_cast<uint8_t*>(p.scales)[go] = (uint8_t)(sbits | (sg ? 0x80u : 0u));
                else
                    reinterpret_cast<uint16_t*>(p.scales)[go] = (uint16_t)(sbits | (sg ? 0x8000u : 0u));
            }
        };
        // Two rows per trip, each in registers of its own: while one is worked on the other's load is in
        // flight, and nothing is copied.  Past the warp's last row the same row is fetched again (unused).
        if (my < N) {
            unsigned wo = (unsigned)my * (unsigned)p.ldw + col_ld, go = (unsigned)my * (unsigned)Gr + col_ld / G;
            unsigned co = ((unsigned)my * (unsigned)K + (unsigned)col0) >> 1;
            uint4 va, vb;
            uint32_t sa, sb;
            load(wo, go, va, sa);
            for (int row = my; row < N; row += 2 * per_slab) {
                const bool more1 = row + per_slab < N;
                const unsigned wo1 = more1 ? wo + step_w : wo, go1 = more1 ? go + step_g : go;
                load(wo1, go1, vb, sb);
                do_row(va, sa, row, go, co);
                if (!more1) break;
                const bool more2 = row + 2 * per_slab < N;
                const unsigned wo2 = more2 ? wo1 + step_w : wo1, go2 = more2 ? go1 + step_g : go1;
                load(wo2, go2, va, sa);
                do_row(vb, sb, row + per_slab, go1, co + step_c);
                wo = wo2; go = go2; co += 2 * step_c;
                nrow += 2;
                if (nrow >= 16) { Eacc += (double)ef; Eout += (double)eof; ef = 0.f; eof = 0.f; nrow = 0; }
            }
        }
        Eacc += (double)ef;
        Eout += (double)eof;
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
    // the last block to finish adds the block partials in block order and hands the results out
    if (tid < 2) {
        double s = 0.0;
        for (unsigned b = 0; b < gridDim.x; ++b) s += __ldcg(p.part + (size_t)b * kPartStride + tid);
        p.ctrl->pack_err[tid] = s;
        if (p.err_out) p.err_out[tid] = s;
    }
    if (tid < 4) {
        if (p.stats) p.stats[tid] = __ldcg(&p.ctrl->pack_stats[tid]);
        p.ctrl->pack_stats[tid] = 0;
    }
    if (tid == 0) p.ctrl->done = 0;
}

template <int MODE, int SEL>
cudaError_t launch_pack_variant(const PackParams& p, unsigned grid, cudaStream_t st) {
    constexpr size_t smem = (size_t)kPackRep * kPackBins * 8 + kLut2Bytes;
    constexpr int kPackWarps = pack_warps(MODE);
    auto kern = pack_kernel<MODE, SEL, kPackWarps, kPackRep>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, kPackWarps * 32, smem, st>>>(p);
    note_launch();
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
    p.err_out = err_out; p.stats = stats;
    if (N > 0x7FFFFFFF || K > 0x7FFFFFFF) return cudaErrorInvalidValue;
    // two blocks per SM; no more warps than there are (row, slab) pieces of work
    const int64_t slabs = (K + 255) / 256;
    int64_t grid = (int64_t)sm_count() * kPackBlocksPerSM;
    const int64_t pieces = (N * slabs + pack_warps(mode) - 1) / pack_warps(mode);
    if (grid > pieces) grid = pieces;
    if (grid > kMaxBlocks) grid = kMaxBlocks;
    if (grid < 1) grid = 1;
    cudaError_t e;
    if (mode == AAAC_INT4 && sel_group == 16) e = launch_pack_variant<AAAC_INT4, 16>(p, (unsigned)grid, st);
    else if (mode == AAAC_INT4) e = launch_pack_variant<AAAC_INT4, 128>(p, (unsigned)grid, st);
    else e = launch_pack_variant<AAAC_NVFP4, 16>(p, (unsigned)grid, st);
    return e;
}

}  // namespace aaac
