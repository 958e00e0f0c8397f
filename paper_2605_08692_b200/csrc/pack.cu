// The final pack pass (Algorithm 1 lines 17-20): BF16 tables, exact selection, 4-bit codes.
//
// For every weight it forms w~ = fl32(w * r) (Eq. 2), finds the interval J of the merged
// breakpoint list of both tables that holds w~, and from J the nearest entry of T0 and of T1
// (Eq. 4).  Per group it sums the two activation-weighted errors (Eq. 8), picks sigma, writes
// the 4-bit codes under the chosen table (Eq. 6) and sigma into the sign bit of the scale.
// (The template keeps a FIT variant of the same loop, which the fit rounds no longer use; the
// round kernel lives in fit.cu.)
//
// Merged breakpoints.  With sorted tables the nearest entry of table r is
// #{i : w~ > mid_r,i}, mid_r,i = (T_r[i] + T_r[i+1]) / 2, and for a float x and a real m,
// x > m  <=>  x > round_down_fp32(m).  The 30 rounded midpoints of both tables are sorted into
// bp[0..29]; J(x) = #{j : bp[j] < x} in 0..30 determines both indices.  J is found from a
// 1025-entry byte table over uniform bins of width 1/64 on (-8, 8) giving the number of
// breakpoints below the bin's lower edge, followed by compares against the next breakpoints.
//
// Exactness of sigma.  The FP32 group errors decide sigma unless |E1 - E0| <= 2^-14 (E0 + E1);
// such groups are re-evaluated in double in index order with the same operations a plain
// double-precision loop uses, so sigma equals the double-precision decision.
//
// Thread mapping.  A block works on items of 32 rows x 256 columns; each of its 8 warps takes
// 4 rows, each lane 8 adjacent columns (one 128-bit load per row).  A group is 2 lanes
// (g = 16) or 16 lanes (g = 128); group sums are xor-shuffle reductions.
#include "internal.cuh"

namespace aaac {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kRowsPerWarp = 4;
constexpr int kRowsPerItem = kWarps * kRowsPerWarp;
constexpr int kNBins = 1025;
constexpr float kMagic = 12582912.f + 512.f;      // 1.5 * 2^23 + 512
constexpr int kMagicBits = 0x4B400000;            // bits of 1.5 * 2^23

struct Luts {
    double Td[2 * kM];
    float bp[32];                 // sorted breakpoints, bp[30] = bp[31] = +inf
    float P[32], Q[32];           // nearest entry of T0 / T1 on interval J
    float rlut[128];              // NVFP4: fl32(1 / s_eff) per E4M3 code
    float slut[128];              // NVFP4: s_eff per E4M3 code
    float tmp_b[32];
    uint8_t tmp_src[32], tmp_exact[32];
    uint8_t src[32], exact[32];   // table of origin; breakpoint is an exact midpoint of two different entries
    uint8_t idx0[32], idx1[32];   // canonical (lowest duplicate) entry index on interval J
    uint8_t clut[kNBins + 3];
    double wsum[kWarps][kPartStride];
    double tot[kPartStride];
    int is_last;
};

struct Params {
    const uint16_t* W;
    int64_t N, K, ldw;
    const void* scales_in;        // FIT: positive scales (NVFP4 bytes); PACK: scales in/out
    void* scales_out;
    const float* rinv;            // FIT INT4
    const float* I;
    const float* tensor_scale;    // PACK NVFP4
    Ctrl* ctrl;
    double* part;
    double* err_slot;
    const float* T01_f32;         // PACK
    uint16_t* T01_bf16;
    uint8_t* codes;
    int64_t items;
    int slabs;
};

__device__ __forceinline__ void sort16(double* t) {
    for (int i = 1; i < kM; ++i) {
        double v = t[i];
        int j = i - 1;
        while (j >= 0 && t[j] > v) { t[j + 1] = t[j]; --j; }
        t[j + 1] = v;
    }
}

template <int MODE, bool PACK>
__device__ void build_luts(Luts& L, const Params& p) {
    const int tid = threadIdx.x;
    if (tid < 2 * kM) {
        if (PACK) {
            const uint32_t b = f32_to_bf16_rne(p.T01_f32[tid]);
            L.Td[tid] = (double)__uint_as_float(b << 16);
        } else {
            L.Td[tid] = p.ctrl->T[tid];
        }
    }
    __syncthreads();
    if (PACK && tid < 2) sort16(L.Td + tid * kM);
    __syncthreads();
    if (PACK && blockIdx.x == 0 && tid < 2 * kM) p.T01_bf16[tid] = (uint16_t)(__float_as_uint((float)L.Td[tid]) >> 16);
    if (tid < kNBP) {
        const int r = tid / 15, i = tid % 15;
        const double a = L.Td[r * kM + i], b = L.Td[r * kM + i + 1];
        const double mid = (a + b) * 0.5;
        const float f = f32_round_down(mid);
        L.tmp_b[tid] = f;
        L.tmp_src[tid] = (uint8_t)r;
        L.tmp_exact[tid] = (uint8_t)(((double)f == mid) && (a != b));
    }
    if (tid >= 30 && tid < 32) L.bp[tid] = __int_as_float(0x7F800000);
    __syncthreads();
    if (tid < kNBP) {
        const float b = L.tmp_b[tid];
        int rank = 0;
        for (int j = 0; j < kNBP; ++j) rank += (L.tmp_b[j] < b) || (L.tmp_b[j] == b && j < tid);
        L.bp[rank] = b;
        L.src[rank] = L.tmp_src[tid];
        L.exact[rank] = L.tmp_exact[tid];
    }
    if (MODE == AAAC_NVFP4 && tid >= 128 && tid < 256) {
        const int c = tid - 128;
        const float s_t = PACK ? p.tensor_scale[0] : p.ctrl->s_t;
        const float s = __fmul_rn(e4m3_value((uint32_t)c), s_t);
        L.slut[c] = s;
        L.rlut[c] = c ? __frcp_rn(s) : 0.f;
    }
    __syncthreads();
    if (tid < kNJ) {
        int i0 = 0, i1 = 0;
        for (int j = 0; j < tid; ++j) { i0 += (L.src[j] == 0); i1 += (L.src[j] == 1); }
        while (i0 > 0 && L.Td[i0 - 1] == L.Td[i0]) --i0;
        while (i1 > 0 && L.Td[kM + i1 - 1] == L.Td[kM + i1]) --i1;
        L.idx0[tid] = (uint8_t)i0;
        L.idx1[tid] = (uint8_t)i1;
        L.P[tid] = (float)L.Td[i0];
        L.Q[tid] = (float)L.Td[kM + i1];
    }
    for (int b = tid; b < kNBins; b += kThreads) {
        const float edge = ((float)b - 512.5f) * 0.015625f;    // lower edge of the bin, exact
        int c = 0;
        for (int j = 0; j < kNBP; ++j) c += (L.bp[j] < edge);
        L.clut[b] = (uint8_t)c;
    }
    __syncthreads();
}

// index of the nearest entry in double, lowest index on ties
__device__ __forceinline__ int nearest_d(const double* T, double x) {
    int best = 0;
    double bd = fabs(__dsub_rn(x, T[0]));
#pragma unroll 1
    for (int i = 1; i < kM; ++i) {
        const double d = fabs(__dsub_rn(x, T[i]));
        if (d < bd) { bd = d; best = i; }
    }
    return best;
}

// Double-precision evaluation of Eq. 8 for the groups whose lanes have need != 0.  Terms are
// I * (d * d) with d = w~ - T[nearest], added in index order.  Every lane of the warp calls this.
template <int LPG>
__device__ void exact_groups(const Luts& L, const float (&x)[8], const float (&Iv)[8], int lane, bool need,
                             bool& sigma, double& emin, bool& tie) {
    unsigned mask = __ballot_sync(0xFFFFFFFFu, need);
    while (mask) {
        const int gbase = (__ffs(mask) - 1) & ~(LPG - 1);
        const bool mine = (lane & ~(LPG - 1)) == gbase;
        double t0[8], t1[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            t0[j] = 0.0;
            t1[j] = 0.0;
            if (mine) {
                const double xd = (double)x[j], id = (double)Iv[j];
                const double d0 = __dsub_rn(xd, L.Td[nearest_d(L.Td, xd)]);
                const double d1 = __dsub_rn(xd, L.Td[kM + nearest_d(L.Td + kM, xd)]);
                t0[j] = __dmul_rn(id, __dmul_rn(d0, d0));
                t1[j] = __dmul_rn(id, __dmul_rn(d1, d1));
            }
        }
        double E0 = 0.0, E1 = 0.0;
        for (int l = 0; l < LPG; ++l) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                E0 = __dadd_rn(E0, __shfl_sync(0xFFFFFFFFu, t0[j], gbase + l));
                E1 = __dadd_rn(E1, __shfl_sync(0xFFFFFFFFu, t1[j], gbase + l));
            }
        }
        if (mine) {
            sigma = E1 < E0;
            emin = sigma ? E1 : E0;
            tie = (E0 == E1);
        }
        mask &= ~(((LPG == 32) ? 0xFFFFFFFFu : ((1u << LPG) - 1u)) << gbase);
    }
}

template <int MODE, bool PACK>
__global__ void __launch_bounds__(kThreads, 1) fit_kernel(const Params p) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    constexpr int LPG = G / 8;
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    __shared__ Luts L;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    build_luts<MODE, PACK>(L, p);

    float2* bins = reinterpret_cast<float2*>(dyn_smem) + (size_t)warp * (2 * kNJ * 32) + lane;
    if (!PACK) {
        for (int b = 0; b < 2 * kNJ; ++b) bins[b * 32] = make_float2(0.f, 0.f);
    }
    double Eacc = 0.0, Eout = 0.0;
    uint32_t n_sig_tie = 0, n_idx_tie = 0, n_exact = 0;
    const int64_t Gr = p.K / G;

    for (int64_t item = blockIdx.x; item < p.items; item += gridDim.x) {
        const int slab = (int)(item % p.slabs);
        const int64_t row0 = (item / p.slabs) * kRowsPerItem + warp * kRowsPerWarp;
        const int64_t col0 = (int64_t)slab * 256 + lane * 8;
        const bool col_ok = col0 < p.K;
        float Iv[8];
        if (col_ok) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(p.I + col0));
            const float4 b = __ldg(reinterpret_cast<const float4*>(p.I + col0 + 4));
            Iv[0] = a.x; Iv[1] = a.y; Iv[2] = a.z; Iv[3] = a.w;
            Iv[4] = b.x; Iv[5] = b.y; Iv[6] = b.z; Iv[7] = b.w;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) Iv[j] = 0.f;
        }
        uint4 v[kRowsPerWarp];
        float rinv[kRowsPerWarp], sval[kRowsPerWarp];
        uint32_t sbits[kRowsPerWarp];
#pragma unroll
        for (int u = 0; u < kRowsPerWarp; ++u) {
            const int64_t row = row0 + u;
            const bool ok = col_ok && row < p.N;
            v[u] = make_uint4(0, 0, 0, 0);
            rinv[u] = 0.f;
            sval[u] = 0.f;
            sbits[u] = 0;
            if (ok) {
                v[u] = __ldcs(reinterpret_cast<const uint4*>(p.W + row * p.ldw + col0));
                const int64_t gi = row * Gr + col0 / G;
                if (MODE == AAAC_NVFP4) {
                    sbits[u] = reinterpret_cast<const uint8_t*>(p.scales_in)[gi] & 0x7Fu;
                } else if (PACK) {
                    sbits[u] = reinterpret_cast<const uint16_t*>(p.scales_in)[gi] & 0x7FFFu;
                } else {
                    rinv[u] = __ldg(p.rinv + gi);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kRowsPerWarp; ++u) {
            const int64_t row = row0 + u;
            const bool ok = col_ok && row < p.N;
            if (MODE == AAAC_NVFP4) {
                rinv[u] = L.rlut[sbits[u]];
                sval[u] = L.slut[sbits[u]];
            } else if (PACK) {
                sval[u] = __uint_as_float(sbits[u] << 16);
                rinv[u] = ok ? __frcp_rn(sval[u]) : 0.f;
            }
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            float x[8];
            int J[8];
            float e0 = 0.f, e1 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float wf = (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]);
                x[j] = __fmul_rn(wf, rinv[u]);
                int bin = __float_as_int(__fmaf_rn(x[j], 64.f, kMagic)) - kMagicBits;
                bin = min(max(bin, 0), kNBins - 1);
                int Jj = L.clut[bin];
                while (x[j] > L.bp[Jj]) ++Jj;
                J[j] = Jj;
                const float d0 = x[j] - L.P[Jj], d1 = x[j] - L.Q[Jj];
                e0 = __fmaf_rn(__fmul_rn(Iv[j], d0), d0, e0);
                e1 = __fmaf_rn(__fmul_rn(Iv[j], d1), d1, e1);
            }
#pragma unroll
            for (int o = LPG / 2; o; o >>= 1) {
                e0 += __shfl_xor_sync(0xFFFFFFFFu, e0, o);
                e1 += __shfl_xor_sync(0xFFFFFFFFu, e1, o);
            }
            bool sigma = e1 < e0;
            double emin = (double)(sigma ? e1 : e0);
            bool tie = false;
            const bool near = ok && (fabsf(e1 - e0) <= 0x1p-14f * (e0 + e1));
            if (__any_sync(0xFFFFFFFFu, near)) {
                exact_groups<LPG>(L, x, Iv, lane, near, sigma, emin, tie);
                if (near && (lane % LPG) == 0) { ++n_exact; n_sig_tie += tie; }
            }
            if (ok && (lane % LPG) == 0) Eacc += emin;

            if (!PACK) {
                if (ok) {
                    float2* b = bins + (sigma ? kNJ * 32 : 0);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float2 a = b[J[j] * 32];
                        a.x = __fmaf_rn(Iv[j], x[j], a.x);
                        a.y += Iv[j];
                        b[J[j] * 32] = a;
                    }
                }
            } else if (ok) {
                uint32_t word = 0;
                float eo = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int Jj = J[j];
                    const uint32_t idx = sigma ? L.idx1[Jj] : L.idx0[Jj];
                    word |= idx << (4 * j);
                    const float tv = sigma ? L.Q[Jj] : L.P[Jj];
                    const float wf = (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]);
                    const float dw = __fmaf_rn(-tv, sval[u], wf);
                    eo = __fmaf_rn(__fmul_rn(Iv[j], dw), dw, eo);
                    for (int jj = Jj; jj < kNBP && L.bp[jj] == x[j]; ++jj)
                        if (L.src[jj] == (uint8_t)sigma && L.exact[jj]) { ++n_idx_tie; break; }
                }
                Eout += (double)eo;
                *reinterpret_cast<uint32_t*>(p.codes + ((row * p.K + col0) >> 1)) = word;
                if ((lane % LPG) == 0) {
                    const int64_t gi = row * Gr + col0 / G;
                    if (MODE == AAAC_NVFP4)
                        reinterpret_cast<uint8_t*>(p.scales_out)[gi] = (uint8_t)(sbits[u] | (sigma ? 0x80u : 0u));
                    else
                        reinterpret_cast<uint16_t*>(p.scales_out)[gi] = (uint16_t)(sbits[u] | (sigma ? 0x8000u : 0u));
                }
            }
        }
    }

    // ---- block partial ----
    if (!PACK) {
        __syncwarp();
        for (int b = 0; b < 2 * kNJ; ++b) {
            const float2 a = bins[b * 32];
            double sx = (double)a.x, sy = (double)a.y;
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                sx += __shfl_xor_sync(0xFFFFFFFFu, sx, o);
                sy += __shfl_xor_sync(0xFFFFFFFFu, sy, o);
            }
            if (lane == 0) { L.wsum[warp][b] = sx; L.wsum[warp][2 * kNJ + b] = sy; }
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        Eacc += __shfl_xor_sync(0xFFFFFFFFu, Eacc, o);
        Eout += __shfl_xor_sync(0xFFFFFFFFu, Eout, o);
    }
    if (lane == 0) { L.wsum[warp][4 * kNJ] = Eacc; L.wsum[warp][4 * kNJ + 1] = Eout; }
    if (PACK) {
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            n_sig_tie += __shfl_xor_sync(0xFFFFFFFFu, n_sig_tie, o);
            n_idx_tie += __shfl_xor_sync(0xFFFFFFFFu, n_idx_tie, o);
            n_exact += __shfl_xor_sync(0xFFFFFFFFu, n_exact, o);
        }
        if (lane == 0) {
            if (n_sig_tie) atomicAdd(&p.ctrl->pack_stats[0], (unsigned long long)n_sig_tie);
            if (n_idx_tie) atomicAdd(&p.ctrl->pack_stats[1], (unsigned long long)n_idx_tie);
            if (n_exact) atomicAdd(&p.ctrl->pack_stats[2], (unsigned long long)n_exact);
        }
    }
    __syncthreads();
    constexpr int kUsed = 4 * kNJ + 2;
    if (tid < kUsed) {
        double s = 0.0;
        const int lo = PACK ? 4 * kNJ : 0;
        if (tid >= lo) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) s += L.wsum[w][tid];
        }
        p.part[(int64_t)blockIdx.x * kPartStride + tid] = s;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) L.is_last = (atomicAdd(&p.ctrl->done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!L.is_last) return;

    // ---- last block: reduce all partials in block order, then update the tables ----
    __threadfence();
    if (tid < kUsed) {
        double s = 0.0;
        for (unsigned b = 0; b < gridDim.x; ++b) s += __ldcg(p.part + (int64_t)b * kPartStride + tid);
        L.tot[tid] = s;
    }
    __syncthreads();
    if (tid == 0) {
        if (!PACK) {
            double S[2 * kM], Wt[2 * kM];
            for (int i = 0; i < 2 * kM; ++i) { S[i] = 0.0; Wt[i] = 0.0; }
            for (int r = 0; r < 2; ++r)
                for (int j = 0; j < kNJ; ++j) {
                    const int i = r * kM + (r ? L.idx1[j] : L.idx0[j]);
                    S[i] += L.tot[r * kNJ + j];
                    Wt[i] += L.tot[2 * kNJ + r * kNJ + j];
                }
            double Tn[2 * kM];
            for (int i = 0; i < 2 * kM; ++i) Tn[i] = (Wt[i] > 0.0) ? __ddiv_rn(S[i], Wt[i]) : L.Td[i];
            sort16(Tn);
            sort16(Tn + kM);
            for (int i = 0; i < 2 * kM; ++i) p.ctrl->T[i] = Tn[i];
            if (p.err_slot) *p.err_slot = L.tot[4 * kNJ];
        } else {
            p.ctrl->pack_err[0] = L.tot[4 * kNJ];
            p.ctrl->pack_err[1] = L.tot[4 * kNJ + 1];
        }
        p.ctrl->done = 0;
    }
}

__global__ void export_pack_kernel(Ctrl* ctrl, double* err_out, unsigned long long* stats) {
    if (threadIdx.x < 2 && err_out) err_out[threadIdx.x] = ctrl->pack_err[threadIdx.x];
    if (threadIdx.x < 4) {
        if (stats) stats[threadIdx.x] = ctrl->pack_stats[threadIdx.x];
        ctrl->pack_stats[threadIdx.x] = 0;
    }
}

}  // namespace

cudaError_t launch_pack(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, const float* I,
                        const float* T01_f32, uint16_t* T01_bf16, void* scales, const float* tensor_scale,
                        uint8_t* codes, double* err_out, unsigned long long* stats, const Workspace& ws,
                        cudaStream_t st) {
    Params p{};
    p.W = W; p.N = N; p.K = K; p.ldw = ldw;
    p.scales_in = scales; p.scales_out = scales; p.I = I; p.tensor_scale = tensor_scale;
    p.ctrl = ws.ctrl; p.part = ws.part; p.T01_f32 = T01_f32; p.T01_bf16 = T01_bf16; p.codes = codes;
    p.slabs = (int)((K + 255) / 256);
    p.items = (int64_t)p.slabs * ((N + kRowsPerItem - 1) / kRowsPerItem);
    int64_t grid = (int64_t)sm_count() * 2;
    if (grid > p.items) grid = p.items;
    if (grid > kMaxBlocks) grid = kMaxBlocks;
    if (mode == AAAC_INT4) fit_kernel<AAAC_INT4, true><<<(unsigned)grid, kThreads, 0, st>>>(p);
    else fit_kernel<AAAC_NVFP4, true><<<(unsigned)grid, kThreads, 0, st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    export_pack_kernel<<<1, 32, 0, st>>>(ws.ctrl, err_out, stats);
    return cudaGetLastError();
}

}  // namespace aaac
