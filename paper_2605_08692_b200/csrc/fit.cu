// One fit round (Algorithm 1 lines 6-16 with n_inner = 1): assignment step (Eq. 8) and
// activation-weighted centroid update (Eq. 11) in a single pass over W.
//
// Per weight the kernel needs (a) the interval J of the merged breakpoint list of both tables
// that holds w~ = fl32(w * r) (Eq. 2) -- J fixes the nearest entry of T0 and of T1 (Eq. 4) --
// (b) its two weighted squared errors, and (c) one accumulation into the centroid sums of cell
// (sigma, J).
//
// (a) Interval.  Uniform bins of width 1/64 on (-8, 8): bin = low 10 bits of
//     fl32(64 x + 1.5 * 2^23 + 512).  A table gives per bin {J_low, thr}: J_low breakpoints lie
//     below the bin, thr is the one breakpoint inside it (+inf if none), J = J_low + (x > thr).
//     Breakpoints are the rounded-down FP32 midpoints, for which x > thr <=> x > midpoint, so J
//     is exact.  A bin that holds two or more breakpoints points at a poisoned slot (J = 31)
//     whose entries are NaN: the group falls through to the exact path below, which searches J
//     directly.  Rows past N are given w~ = NaN, which lands in bin 0 or 1023 (outside the range
//     of w~, always poisoned): their sums go to a slot nobody reads.
// (b) Selection.  A second table gives {P, Q}, the FP32 roundings of the nearest entries of T0
//     and T1 on interval J; u_r = x - T_r, E_r = sum_k I_k u_r^2 (Eq. 8), summed per lane and
//     over the lanes of the group by shuffles; sigma = [E1 < E0].
//     Rounding: with eta = 2^-24 max|T|, |E_r - E_r,exact| <= 2^-24 * 16 E_r + 2 eta sum I |u_r|
//     and sum I |u_r| <= sqrt(sum I * E_r).  Groups with
//     |E0 - E1| <= 2^-24 (16 (E0 + E1) + 2.83 max|T| sqrt(sum I (E0 + E1))) (and NaN) are
//     re-evaluated in double with the unrounded entries, so sigma is the double-precision
//     decision.
// (c) Centroid sums, centred.  Lane-private shared-memory bins [sigma][J] hold
//     (sum I (x - T), sum I) with T the (rounded) entry the weight is assigned to, so the new
//     entry is T + sum I (x - T) / sum I.  The residual sums are small and of mixed sign, which
//     keeps the FP32 accumulation error some 20 times below that of sum I x.  No atomics, fixed
//     order.  One partial per block; the last block to finish adds the partials in block order,
//     forms the centroids, keeps entries of empty cells, sorts, and stores the new tables and
//     the Eq. 8 objective of the round (sum over groups of the smaller error).
//
// Tables in shared memory are replicated so that lookups are free of bank conflicts: the
// {J_low, thr} table once per lane of a half-warp (64-bit accesses are served per half-warp),
// the {P, Q} table and the bins once per lane.
//
// Thread mapping.  A block works on items of 32 rows x 256 columns, dealt to blocks as
// contiguous ranges (slab-major), so every sum has a fixed order and results are bitwise
// reproducible.  A warp takes 32 / NW rows; each lane 8 adjacent columns (one 128-bit load
// per row), so its eight importances stay in registers.  A group is 2 lanes (g = 16) or 16
// lanes (g = 128).  The next item's rows are loaded while the current item is processed.
#include "internal.cuh"

namespace aaac {

namespace {

constexpr int kRowsPerItem = 32;
constexpr int kNBins = 1024;
constexpr int kJSlots = 32;                        // 31 intervals + the poisoned slot
constexpr int kSlotBytes = 32 * 8;                 // one 8-byte entry per lane
constexpr int kPoison = kNJ * kSlotBytes;          // byte offset of the poisoned slot
constexpr float kMagic = 12582912.f + 512.f;       // 1.5 * 2^23 + 512
constexpr int kUsed = 4 * kNJ + 1;                 // [2][31] S, [2][31] Wt, E

// Shared-memory accesses of the hot loop with explicit 32-bit addresses.  The table loads are
// plain asm (the tables are not written while the main loop runs, so they may move freely);
// the bin accesses are volatile, which keeps every read-modify-write in program order.
__device__ __forceinline__ uint2 lds_table_u2(uint32_t addr) {
    uint2 r;
    asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "r"(addr));
    return r;
}
__device__ __forceinline__ float2 lds_table_f2(uint32_t addr) {
    float2 r;
    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(r.x), "=f"(r.y) : "r"(addr));
    return r;
}
__device__ __forceinline__ float2 lds_bin(uint32_t addr) {
    float2 r;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(r.x), "=f"(r.y) : "r"(addr) : "memory");
    return r;
}
__device__ __forceinline__ void sts_bin(uint32_t addr, float2 v) {
    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" :: "r"(addr), "f"(v.x), "f"(v.y) : "memory");
}

struct FitTables {
    double Td[2 * kM];
    double2 PQ[kJSlots];          // nearest entries of T0 / T1 on interval J, as double
    float bp[32];                 // sorted breakpoints, bp[30] = bp[31] = +inf
    float tmp_b[32];
    uint8_t tmp_src[32];
    uint8_t src[32];
    uint8_t idx0[32], idx1[32];   // canonical (lowest duplicate) entry index on interval J
    float rlut[128];              // NVFP4: fl32(1 / s_eff) per E4M3 code; [127] = NaN marks a row past N
    float tmax283;                // 2.83 * max |entry|, rounded up
    int is_last;
};

template <int NW>
struct FitShared {
    FitTables t;
    double wsum[NW][kPartStride];
    double tot[kPartStride];
};

struct FitParams {
    const uint16_t* W;
    int64_t N, K, ldw;
    const uint8_t* scales;        // NVFP4 scale bytes
    const float* rinv;            // INT4 reciprocal scales
    const float* I;
    Ctrl* ctrl;
    double* part;
    double* err_slot;
    int64_t items, per_block, nrb;
};

__device__ __forceinline__ void sort16(double* t) {
    for (int i = 1; i < kM; ++i) {
        double v = t[i];
        int j = i - 1;
        while (j >= 0 && t[j] > v) { t[j + 1] = t[j]; --j; }
        t[j + 1] = v;
    }
}

// Builds every lookup table of the round from the current tables in the control block.
template <int MODE, int NW, int REP>
__device__ void build_tables(FitTables& S, const FitParams& p, unsigned char* dyn) {
    constexpr int NT = NW * 32;
    const int tid = threadIdx.x;
    if (tid < 2 * kM) S.Td[tid] = p.ctrl->T[tid];
    __syncthreads();
    if (tid < kNBP) {
        const int r = tid / 15, i = tid % 15;
        const double mid = (S.Td[r * kM + i] + S.Td[r * kM + i + 1]) * 0.5;
        S.tmp_b[tid] = f32_round_down(mid);
        S.tmp_src[tid] = (uint8_t)r;
    }
    if (tid >= 30 && tid < 32) S.bp[tid] = __int_as_float(0x7F800000);
    if (MODE == AAAC_NVFP4 && tid < 128) {
        const float s = __fmul_rn(e4m3_value((uint32_t)tid), p.ctrl->s_t);
        S.rlut[tid] = tid == 127 ? __int_as_float(0x7FFFFFFF) : (tid ? __frcp_rn(s) : 0.f);
    }
    __syncthreads();
    if (tid < kNBP) {
        const float b = S.tmp_b[tid];
        int rank = 0;
        for (int j = 0; j < kNBP; ++j) rank += (S.tmp_b[j] < b) || (S.tmp_b[j] == b && j < tid);
        S.bp[rank] = b;
        S.src[rank] = S.tmp_src[tid];
    }
    __syncthreads();
    float2* lut2 = reinterpret_cast<float2*>(dyn + (size_t)REP * kNBins * 8);
    if (tid < kJSlots) {
        float P = __int_as_float(0x7FC00000), Q = P;
        if (tid < kNJ) {
            int i0 = 0, i1 = 0;
            for (int j = 0; j < tid; ++j) { i0 += (S.src[j] == 0); i1 += (S.src[j] == 1); }
            while (i0 > 0 && S.Td[i0 - 1] == S.Td[i0]) --i0;
            while (i1 > 0 && S.Td[kM + i1 - 1] == S.Td[kM + i1]) --i1;
            S.idx0[tid] = (uint8_t)i0;
            S.idx1[tid] = (uint8_t)i1;
            S.PQ[tid] = make_double2(S.Td[i0], S.Td[kM + i1]);
            P = (float)S.Td[i0];
            Q = (float)S.Td[kM + i1];
        } else {
            S.PQ[tid] = make_double2(0.0, 0.0);
            S.idx0[tid] = 0;
            S.idx1[tid] = 0;
        }
        double tm = fabs(S.Td[tid]);                     // 32 entries, one per lane of warp 0
#pragma unroll
        for (int o = 16; o; o >>= 1) tm = fmax(tm, __shfl_xor_sync(0xFFFFFFFFu, tm, o));
        if (tid == 0) S.tmax283 = __double2float_ru(tm * 2.83);
        for (int l = 0; l < 32; ++l) lut2[tid * 32 + l] = make_float2(P, Q);
    }
    // {J_low, thr} per bin; bin b holds the x with 64 x + 512 in [b - 1/2, b + 1/2]
    uint2* lut1 = reinterpret_cast<uint2*>(dyn);
    for (int b = tid; b < kNBins; b += NT) {
        const float lo = ((float)b - 512.5f) * 0.015625f, hi = ((float)b - 511.5f) * 0.015625f;
        int below = 0, inside = 0;
        float thr = __int_as_float(0x7F800000);
        for (int j = 0; j < kNBP; ++j) {
            const float v = S.bp[j];
            below += (v < lo);
            if (v >= lo && v <= hi) {
                if (inside == 0) thr = v;
                ++inside;
            }
        }
        uint2 e;
        // bins 0 and 1023 lie outside the range of w~; a NaN (a row past N) lands there
        if (inside <= 1 && b != 0 && b != kNBins - 1) {
            e.x = (uint32_t)(below * kSlotBytes);
            e.y = __float_as_uint(thr);
        } else {
            e.x = (uint32_t)kPoison;
            e.y = 0x7F800000u;
        }
#pragma unroll
        for (int c = 0; c < REP; ++c) lut1[b * REP + c] = e;
    }
    __syncthreads();
}

struct Row8 { float x[8]; float I[8]; int o[8]; };
struct Exact8 { int o[8]; float m0[8], m1[8]; double emin; int sigma; };

// Double-precision decision (Eq. 8 as a plain double-precision loop states it, lanes of a group
// combined by a shuffle tree) for the groups whose lanes pass need != 0; every lane of the warp
// calls.  Poisoned slots are replaced by the interval found by direct search, and the centred
// terms I (x - T) of those weights are formed.
template <int LPG>
__device__ __noinline__ Exact8 exact_groups(const FitTables* S, Row8 r, int c0, int need) {
    Exact8 out;
    double e0 = 0.0, e1 = 0.0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        int o = r.o[j];
        out.m0[j] = 0.f;
        out.m1[j] = 0.f;
        if (need) {
            int J = (o - c0) >> 8;
            if (J >= kNJ) {
                J = 0;
#pragma unroll 1
                for (int i = 0; i < kNBP; ++i) J += (S->bp[i] < r.x[j]);
                o = J * kSlotBytes + c0;
            }
            const double2 pq = S->PQ[J];
            const double xd = (double)r.x[j], id = (double)r.I[j];
            const double d0 = __dsub_rn(xd, pq.x), d1 = __dsub_rn(xd, pq.y);
            e0 = __dadd_rn(e0, __dmul_rn(id, __dmul_rn(d0, d0)));
            e1 = __dadd_rn(e1, __dmul_rn(id, __dmul_rn(d1, d1)));
            out.m0[j] = __fmul_rn(r.I[j], __fsub_rn(r.x[j], (float)pq.x));
            out.m1[j] = __fmul_rn(r.I[j], __fsub_rn(r.x[j], (float)pq.y));
        }
        out.o[j] = o;
    }
#pragma unroll
    for (int s = LPG / 2; s; s >>= 1) {
        e0 = __dadd_rn(e0, __shfl_xor_sync(0xFFFFFFFFu, e0, s));
        e1 = __dadd_rn(e1, __shfl_xor_sync(0xFFFFFFFFu, e1, s));
    }
    out.sigma = e1 < e0;
    out.emin = out.sigma ? e1 : e0;
    return out;
}

template <int MODE, int NW, int REP>
__global__ void __launch_bounds__(NW * 32, 1) fit_round_kernel(const FitParams p) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    constexpr int LPG = G / 8;
    constexpr int R = kRowsPerItem / NW;
    constexpr int kLut1Bytes = REP * kNBins * 8;
    constexpr int kLut2Bytes = kJSlots * kSlotBytes;
    constexpr int kBinBytes = 2 * kJSlots * kSlotBytes;      // per warp
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ FitShared<NW> S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    build_tables<MODE, NW, REP>(S.t, p, dyn);

    // 32-bit shared addresses.  Slot offsets carry the address of this lane's column of the
    // {P, Q} table, so a lookup there needs no further arithmetic; the bins of (warp, sigma) lie
    // at a fixed distance from it.
    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(dyn);
    const uint32_t lut1_lane = sm_base + (lane & (REP - 1)) * 8;                       // + bin * REP * 8
    const int c0 = (int)(sm_base + kLut1Bytes + lane * 8), c1 = c0 + kSlotBytes;       // + J * 256
    const uint32_t bins_rel = kLut2Bytes + warp * kBinBytes;                           // + sigma * 8192
    for (int b = 0; b < 2 * kJSlots; ++b) sts_bin((uint32_t)c0 + bins_rel + b * kSlotBytes, make_float2(0.f, 0.f));
    const float tmax283 = S.t.tmax283;
    double Eacc = 0.0;

    const int64_t Gr = p.K / G;
    const int64_t it0 = (int64_t)blockIdx.x * p.per_block;
    const int64_t it1 = min(p.items, it0 + p.per_block);

    uint4 nv[R];
    uint32_t ns[R];           // NVFP4: scale byte; INT4: bits of the reciprocal scale
    auto load_item = [&](int64_t item) {
        const int64_t slab = item / p.nrb, rb = item - slab * p.nrb;
        const int64_t col0 = slab * 256 + lane * 8;
        const int64_t row0 = rb * kRowsPerItem + warp * R;
#pragma unroll
        for (int u = 0; u < R; ++u) {
            const int64_t row = row0 + u;
            nv[u] = make_uint4(0, 0, 0, 0);
            ns[u] = row < p.N ? 0u : (MODE == AAAC_NVFP4 ? 0x7Fu : 0x7FFFFFFFu);   // past N: w~ = NaN
            if (col0 < p.K && row < p.N) {
                nv[u] = __ldcs(reinterpret_cast<const uint4*>(p.W + row * p.ldw + col0));
                const int64_t gi = row * Gr + col0 / G;
                if (MODE == AAAC_NVFP4) ns[u] = p.scales[gi];      // masked at use: nothing waits on the load here
                else ns[u] = __float_as_uint(__ldg(p.rinv + gi));
            }
        }
    };

    int64_t cur_slab = -1;
    float Iv[8];
    float isum = 0.f;         // sum of I over the lane's group (rounded up a little)
    bool col_ok = false;
#pragma unroll
    for (int j = 0; j < 8; ++j) Iv[j] = 0.f;

    if (it0 < it1) load_item(it0);
    for (int64_t item = it0; item < it1; ++item) {
        uint4 v[R];
        uint32_t sc[R];
#pragma unroll
        for (int u = 0; u < R; ++u) { v[u] = nv[u]; sc[u] = ns[u]; }
        if (item + 1 < it1) load_item(item + 1);

        const int64_t slab = item / p.nrb, rb = item - slab * p.nrb;
        if (slab != cur_slab) {
            cur_slab = slab;
            const int64_t col0 = slab * 256 + lane * 8;
            col_ok = col0 < p.K;
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
        const int64_t row0 = rb * kRowsPerItem + warp * R;

        // Two rows are in flight: m = I (x - T_sigma) and the slot offsets of the row whose bins
        // are being updated, and the lookups of the next row.
        float m[2][8];
        int o[2][8];
        bool sigma[2] = {false, false};

        // lookups and both weighted errors of row u; decides sigma, leaves the centred terms
        auto stage_a = [&](int u, float (&ms)[8], int (&os)[8], bool& sg) {
            const float rinv = MODE == AAAC_NVFP4 ? S.t.rlut[sc[u] & 0x7Fu] : __uint_as_float(sc[u]);
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            float xs[8], m0[8], m1[8];
            float e0 = 0.f, e1 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float wf = (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]);
                xs[j] = __fmul_rn(wf, rinv);
                const uint32_t bin = (uint32_t)__float_as_int(__fmaf_rn(xs[j], 64.f, kMagic)) & (kNBins - 1);
                const uint2 e = lds_table_u2(lut1_lane + bin * (REP * 8));
                os[j] = (int)e.x + ((xs[j] > __uint_as_float(e.y)) ? c1 : c0);
                const float2 pq = lds_table_f2((uint32_t)os[j]);
                const float u0 = __fsub_rn(xs[j], pq.x), u1 = __fsub_rn(xs[j], pq.y);
                m0[j] = __fmul_rn(Iv[j], u0);
                m1[j] = __fmul_rn(Iv[j], u1);
                e0 = __fmaf_rn(m0[j], u0, e0);
                e1 = __fmaf_rn(m1[j], u1, e1);
            }
#pragma unroll
            for (int s = LPG / 2; s; s >>= 1) {
                e0 += __shfl_xor_sync(0xFFFFFFFFu, e0, s);
                e1 += __shfl_xor_sync(0xFFFFFFFFu, e1, s);
            }
            const bool ok = col_ok && (row0 + u) < p.N;
            const float es = e0 + e1;
            const float tau = 0x1p-24f * __fmaf_rn(tmax283, __fsqrt_ru(__fmul_ru(isum, es)), 16.f * es);
            const bool near = ok && !(fabsf(e1 - e0) > tau);
            sg = e1 < e0;
            double emin = (double)(sg ? e1 : e0);
            if (__any_sync(0xFFFFFFFFu, near)) {
                Row8 r;
#pragma unroll
                for (int j = 0; j < 8; ++j) { r.x[j] = xs[j]; r.I[j] = Iv[j]; r.o[j] = os[j]; }
                const Exact8 ex = exact_groups<LPG>(&S.t, r, c0, (int)near);
                if (near) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) { os[j] = ex.o[j]; m0[j] = ex.m0[j]; m1[j] = ex.m1[j]; }
                    sg = ex.sigma != 0;
                    emin = ex.emin;
                }
            }
            if (ok && (lane % LPG) == 0) Eacc += emin;
#pragma unroll
            for (int j = 0; j < 8; ++j) ms[j] = sg ? m1[j] : m0[j];
        };
        // centroid sums of one row
        auto stage_b = [&](const float (&ms)[8], const int (&os)[8], bool sg) {
            const uint32_t rel = bins_rel + (sg ? kJSlots * kSlotBytes : 0);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t addr = (uint32_t)os[j] + rel;
                float2 a = lds_bin(addr);
                a.x += ms[j];
                a.y += Iv[j];
                sts_bin(addr, a);
            }
        };

        // Software-pipelined: the lookups of row u + 1 are issued before the read-modify-write
        // chain of row u.
        stage_a(0, m[0], o[0], sigma[0]);
#pragma unroll
        for (int u = 0; u < R; ++u) {
            const int cur = u & 1, nxt = cur ^ 1;
            if (u + 1 < R) stage_a(u + 1, m[nxt], o[nxt], sigma[nxt]);
            stage_b(m[cur], o[cur], sigma[cur]);
        }
    }

    // ---- block partial: add the lanes of every bin, then the warps ----
    __syncwarp();
    for (int b = 0; b < 2 * kNJ; ++b) {
        const int sg = b / kNJ, J = b - sg * kNJ;
        const float2 a = lds_bin((uint32_t)c0 + bins_rel + (sg * kJSlots + J) * kSlotBytes);
        double sx = (double)a.x, sy = (double)a.y;
#pragma unroll
        for (int s = 16; s; s >>= 1) {
            sx += __shfl_xor_sync(0xFFFFFFFFu, sx, s);
            sy += __shfl_xor_sync(0xFFFFFFFFu, sy, s);
        }
        if (lane == 0) { S.wsum[warp][b] = sx; S.wsum[warp][2 * kNJ + b] = sy; }
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) Eacc += __shfl_xor_sync(0xFFFFFFFFu, Eacc, s);
    if (lane == 0) S.wsum[warp][4 * kNJ] = Eacc;
    __syncthreads();
    if (tid < kUsed) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < NW; ++w) s += S.wsum[w][tid];
        p.part[(int64_t)blockIdx.x * kPartStride + tid] = s;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) S.t.is_last = (atomicAdd(&p.ctrl->done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!S.t.is_last) return;

    // ---- last block: add the partials in block order, then update the tables ----
    __threadfence();
    if (tid < kUsed) {
        double s = 0.0;
        for (unsigned b = 0; b < gridDim.x; ++b) s += __ldcg(p.part + (int64_t)b * kPartStride + tid);
        S.tot[tid] = s;
    }
    __syncthreads();
    if (tid == 0) {
        double Sx[2 * kM], Wt[2 * kM];
        for (int i = 0; i < 2 * kM; ++i) { Sx[i] = 0.0; Wt[i] = 0.0; }
        for (int r = 0; r < 2; ++r)
            for (int j = 0; j < kNJ; ++j) {
                const int i = r * kM + (r ? S.t.idx1[j] : S.t.idx0[j]);
                Sx[i] += S.tot[r * kNJ + j];
                Wt[i] += S.tot[2 * kNJ + r * kNJ + j];
            }
        double Tn[2 * kM];
        for (int i = 0; i < 2 * kM; ++i) {
            // the sums are centred on the FP32 rounding of the entry
            const double c = (double)(float)S.t.Td[i];
            Tn[i] = (Wt[i] > 0.0) ? c + __ddiv_rn(Sx[i], Wt[i]) : S.t.Td[i];
        }
        sort16(Tn);
        sort16(Tn + kM);
        for (int i = 0; i < 2 * kM; ++i) p.ctrl->T[i] = Tn[i];
        if (p.err_slot) *p.err_slot = S.tot[4 * kNJ];
        p.ctrl->done = 0;
    }
}

__global__ void export_tables_kernel(const Ctrl* ctrl, float* T01) {
    if (threadIdx.x < 2 * kM) T01[threadIdx.x] = (float)ctrl->T[threadIdx.x];
}

template <int MODE, int NW, int REP>
cudaError_t launch_variant(const FitParams& p, unsigned grid, cudaStream_t st) {
    constexpr size_t smem = (size_t)REP * kNBins * 8 + kJSlots * kSlotBytes + (size_t)NW * 2 * kJSlots * kSlotBytes;
    auto kern = fit_round_kernel<MODE, NW, REP>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, NW * 32, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fit_round(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, const void* scales,
                             const float* I, double* err_slot, const Workspace& ws, cudaStream_t st) {
    FitParams p{};
    p.W = W; p.N = N; p.K = K; p.ldw = ldw;
    p.scales = static_cast<const uint8_t*>(scales); p.rinv = ws.rinv; p.I = I;
    p.ctrl = ws.ctrl; p.part = ws.part; p.err_slot = err_slot;
    const int64_t slabs = (K + 255) / 256;
    p.nrb = (N + kRowsPerItem - 1) / kRowsPerItem;
    p.items = slabs * p.nrb;
    int64_t grid = sm_count();
    if (grid > p.items) grid = p.items;
    if (grid > kMaxBlocks) grid = kMaxBlocks;
    p.per_block = (p.items + grid - 1) / grid;
    grid = (p.items + p.per_block - 1) / p.per_block;
    constexpr int NW = AAAC_FIT_WARPS, REP = AAAC_FIT_REP;
    if (mode == AAAC_INT4) return launch_variant<AAAC_INT4, NW, REP>(p, (unsigned)grid, st);
    return launch_variant<AAAC_NVFP4, NW, REP>(p, (unsigned)grid, st);
}

cudaError_t launch_export_tables(float* T01, const Workspace& ws, cudaStream_t st) {
    export_tables_kernel<<<1, 32, 0, st>>>(ws.ctrl, T01);
    return cudaGetLastError();
}

}  // namespace aaac
