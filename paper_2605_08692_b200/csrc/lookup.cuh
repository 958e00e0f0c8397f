// Lookup machinery shared by the fit rounds (fit.cu) and the pack pass (pack.cu): the tables that
// turn a normalised weight into its interval of the merged breakpoint list and into the nearest
// entries of T0 and T1, their construction, and the double-precision fallback.  See the header
// comment of fit.cu for the method.
#pragma once
#include "internal.cuh"

namespace aaac {

constexpr int kRowsPerWarp = 4;
constexpr int kNBins = 1024;                       // default number of uniform bins on (-8, 8): width 1/64
constexpr int kJSlots = 32;                        // 31 intervals + the poisoned slot
constexpr int kSlotBytes = 32 * 8;                 // bytes of a lane-private bin slot (one 8-byte entry per lane)
// The {P, Q} table: one 256-byte pair per interval J -- entry J in 16 columns of 8 bytes, then
// entry J + 1 in 16 columns -- so that a bin's table entry can name the address of its lower
// interval and a weight above the bin's breakpoint adds kPairHalf to it.  Lane l uses column
// l mod 16: an 8-byte load is served a half-warp at a time, so lanes l and l + 16 never meet.
constexpr int kPairBytes = 256;
constexpr int kPairHalf = 128;
constexpr int kPqCols = 16;
constexpr int kPoison = kNJ * kPairBytes;          // byte offset of the poisoned pair (both halves NaN)
constexpr int kLut2Bytes = kJSlots * kPairBytes;
constexpr int kCells = 2 * kM;                     // bins per lane: [sigma][entry]
constexpr int kUsed = 2 * kCells + 1;              // [32] S, [32] Wt, E
constexpr uint32_t kIdxMask = 15u;                 // low mantissa bits of a centre constant = entry index

// Shared-memory accesses of the hot loop with explicit 32-bit addresses.  All are volatile asm,
// which keeps them in the order in which the loop writes them (table lookups of one row issued
// ahead of the read-modify-write chain of the previous one).
__device__ __forceinline__ uint2 lds_table_u2(uint32_t addr) {
    uint2 r;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "r"(addr));
    return r;
}
__device__ __forceinline__ float2 lds_table_f2(uint32_t addr) {
    float2 r;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(r.x), "=f"(r.y) : "r"(addr));
    return r;
}
__device__ __forceinline__ uint64_t lds_table_b64(uint32_t addr) {
    uint64_t r;
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(r) : "r"(addr));
    return r;
}

// Packed pairs of FP32 values in one 64-bit register and the two-wide FP32 instructions of
// sm_100 on them (each half is rounded exactly like the scalar instruction).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ float lo2(uint64_t v) { float lo, hi; unpack2(v, lo, hi); return lo; }
__device__ __forceinline__ float hi2(uint64_t v) { float lo, hi; unpack2(v, lo, hi); return hi; }
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// {x - P, x - Q}: each half one correctly rounded FP32 subtraction, either as two scalar
// instructions writing a register pair or as one packed instruction on {x, x}
#ifndef AAAC_SCALAR_SUB
#define AAAC_SCALAR_SUB 1
#endif
__device__ __forceinline__ uint64_t diff2(float x, uint64_t pq) {
#if AAAC_SCALAR_SUB
    float P, Q;
    unpack2(pq, P, Q);
    return pack2(__fsub_rn(x, P), __fsub_rn(x, Q));
#else
    return sub2(pack2(x, x), pq);
#endif
}

// Address of the {P, Q} entry of a weight: `a` names the entry of the lower interval of the
// weight's bin; a weight above the bin's breakpoint belongs to the next interval, whose entry
// lies kPairHalf bytes further (one compare and one predicated add).
__device__ __forceinline__ uint32_t above_addr(uint32_t a, float x, uint32_t thr_bits) {
    asm("{\n\t.reg .pred p;\n\tsetp.gt.f32 p, %1, %2;\n\t@p add.u32 %0, %0, 128;\n\t}"
        : "+r"(a) : "f"(x), "f"(__uint_as_float(thr_bits)));
    return a;
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
    uint8_t src[32];              // table a breakpoint comes from
    uint8_t tmp_exact[32], exact[32];   // the breakpoint is the exact midpoint of two different entries
    float rlut[128];              // NVFP4: fl32(1 / s_eff) per E4M3 code
    float2 pq32[kJSlots];         // {P, Q} of every interval before replication
    float centre[2 * kM];         // centre constant of every entry (index in the low 4 mantissa bits)
    float tmax283;                // 2.83 * 17 * max |entry|, rounded up
    int no_dup;                   // no table holds two equal entries: the interval of a weight is then the sum of its two entry indices
    int is_last;
    double tot[kPartStride];
    double fix_scale, fix_unscale;   // fit rounds: fixed-point scale of the sums over the blocks and its inverse
};

// Builds every lookup table of the round from the current tables in S.Td.
template <int MODE, int NW, int REP, int NB = kNBins>
__device__ void build_tables(FitTables& S, unsigned char* lut1_mem, unsigned char* lut2_mem) {
    constexpr int NT = NW * 32;
    const int tid = threadIdx.x;
    if (tid < kNBP) {
        const int r = tid / 15, i = tid % 15;
        const double mid = (S.Td[r * kM + i] + S.Td[r * kM + i + 1]) * 0.5;
        const float f = f32_round_down(mid);
        S.tmp_b[tid] = f;
        S.tmp_src[tid] = (uint8_t)r;
        S.tmp_exact[tid] = (uint8_t)(((double)f == mid) && (S.Td[r * kM + i] != S.Td[r * kM + i + 1]));
    }
    if (tid >= 30 && tid < 32) S.bp[tid] = __int_as_float(0x7F800000);
    if (tid >= 32 && tid < 32 + 2 * kM) {
        // centre constant: close to the FP32 rounding of the entry, with the entry's canonical
        // (lowest duplicate) index in the low mantissa bits
        const int t = tid - 32, r = t & 16;
        int i = t & 15;
        while (i > 0 && S.Td[r + i - 1] == S.Td[r + i]) --i;
        // the float nearest to the FP32 rounding of the entry whose low 4 mantissa bits are i
        // (at most 8 units in the last place away)
        const uint32_t b = __float_as_uint((float)S.Td[t]);
        const int mag = (int)(b & 0x7FFFFFFFu);
        const int tt = mag + 8 - i;
        const uint32_t mag2 = tt < 0 ? (uint32_t)i : (uint32_t)((tt & ~15) + i);
        S.centre[t] = __uint_as_float((b & 0x80000000u) | mag2);
        const bool all_distinct = __all_sync(0xFFFFFFFFu, i == (t & 15));      // threads 32..63 are one warp
        if (t == 0) S.no_dup = all_distinct;
    }
    __syncthreads();
    if (tid < kNBP) {
        const float b = S.tmp_b[tid];
        int rank = 0;
        for (int j = 0; j < kNBP; ++j) rank += (S.tmp_b[j] < b) || (S.tmp_b[j] == b && j < tid);
        S.bp[rank] = b;
        S.src[rank] = S.tmp_src[tid];
        S.exact[rank] = S.tmp_exact[tid];
    }
    __syncthreads();
    float2* lut2 = reinterpret_cast<float2*>(lut2_mem);
    if (tid < kJSlots) {
        float P = __int_as_float(0x7FC00000), Q = P;
        if (tid < kNJ) {
            // entries of T0 / T1 whose upper midpoint lies below interval tid
            const unsigned from1 = __ballot_sync(0x7FFFFFFFu, tid < kNBP && S.src[tid] == 1);
            int i1 = __popc(from1 & ((1u << tid) - 1u)), i0 = tid - i1;
            while (i0 > 0 && S.Td[i0 - 1] == S.Td[i0]) --i0;
            while (i1 > 0 && S.Td[kM + i1 - 1] == S.Td[kM + i1]) --i1;
            S.PQ[tid] = make_double2(S.Td[i0], S.Td[kM + i1]);
            P = S.centre[i0];
            Q = S.centre[kM + i1];
        } else {
            S.PQ[tid] = make_double2(0.0, 0.0);
        }
        double tm = fabs(S.Td[tid]);                     // 32 entries, one per lane of warp 0
#pragma unroll
        for (int o = 16; o; o >>= 1) tm = fmax(tm, __shfl_xor_sync(0xFFFFFFFFu, tm, o));
        if (tid == 0) S.tmax283 = __double2float_ru(tm * (2.83 * 17.0));
        S.pq32[tid] = make_float2(P, Q);
    }
    // {slot address, thr} per bin.  With s = NB / 16 bins per unit, bin b holds the x with s x + NB / 2 in
    // [b - h, b + 1 - h], h = half of the rounding step 1 / (8 REP) of the bin arithmetic.  The breakpoints are sorted, so those
    // inside a bin are the first ones not below its lower edge.  The entries are first written
    // once per bin (into the space of the {P, Q} table, which is filled afterwards) and then
    // replicated REP times by consecutive lanes writing consecutive addresses: both steps are free
    // of bank conflicts (one thread writing the REP copies of its bin would serialise 32-fold).
    static_assert(NB * 8 <= kLut2Bytes, "the per-bin entries are staged in the {P, Q} table's space");
    static_assert(REP == kPqCols, "copy c of a bin's entry carries the address of column c of the {P, Q} table");
    uint2* binval = reinterpret_cast<uint2*>(lut2_mem);
    const uint32_t lut2_addr = (uint32_t)__cvta_generic_to_shared(lut2_mem);
    constexpr float h = 0.5f / (float)(REP * 8);
    constexpr float kHalf = (float)(NB / 2), kWidth = 16.f / (float)NB;
    for (int b = tid; b < NB; b += NT) {
        const float lo = ((float)b - kHalf - h) * kWidth, hi = ((float)b - (kHalf - 1.f) - h) * kWidth;
        int below = 0;                                   // number of breakpoints < lo (binary search)
#pragma unroll
        for (int step = 16; step; step >>= 1)
            if (below + step <= kNBP && S.bp[below + step - 1] < lo) below += step;
        const float v0 = S.bp[below], v1 = S.bp[below + 1];     // bp[30], bp[31] = +inf
        uint2 e;
        if (!(v1 <= hi)) {                               // at most one breakpoint inside
            e.x = lut2_addr + (uint32_t)(below * kPairBytes);
            e.y = v0 <= hi ? __float_as_uint(v0) : 0x7F800000u;
        } else {
            e.x = lut2_addr + (uint32_t)kPoison;
            e.y = 0x7F800000u;
        }
        binval[b] = e;
    }
    __syncthreads();
    {
        uint4* lut1v = reinterpret_cast<uint4*>(lut1_mem);    // two copies (columns 2 i mod REP and the next) per store
        for (int i = tid; i < NB * REP / 2; i += NT) {
            const uint2 e = binval[(2 * i) / REP];
            const uint32_t col = (uint32_t)((2 * i) % REP) * 8u;
            lut1v[i] = make_uint4(e.x + col, e.y, e.x + col + 8u, e.y);
        }
    }
    __syncthreads();
    // pair J = {entry J, entry J + 1}, 16 columns each; the pair after the last interval is the poisoned one
    for (int i = tid; i < kJSlots * 32; i += NT) {
        const int pair = i >> 5, half = (i >> 4) & 1;
        const int J = pair < kNJ ? min(pair + half, kNJ - 1) : kNJ;      // kNJ: the NaN entry
        lut2[i] = S.pq32[J];
    }
    __syncthreads();
}

// the two tables one after the other in one buffer
template <int MODE, int NW, int REP, int NB = kNBins>
__device__ __forceinline__ void build_tables(FitTables& S, unsigned char* dyn) {
    build_tables<MODE, NW, REP, NB>(S, dyn, dyn + (size_t)REP * NB * 8);
}

// address of column (lane mod 16) of interval J's entry in the {P, Q} table that starts at lut2_addr
__device__ __forceinline__ uint32_t pq_entry_addr(uint32_t lut2_addr, int J, int lane) {
    return lut2_addr + (uint32_t)(J * kPairBytes) + (uint32_t)(lane & (kPqCols - 1)) * 8u;
}

// hint[j] < kNJ names the interval of weight j where the caller knows it, else the interval is searched
struct Row8 { float x[8]; float I[8]; uint32_t hint[8]; };
constexpr uint32_t kNoHint = 0xFFu;

// The interval of a weight from the constants {P, Q} the fast path has looked up: with no equal
// entries inside a table, entry index = number of that table's breakpoints below the weight, and
// the interval of the merged list is the sum of the two.  (A poisoned slot reads as NaN: no hint.)
#ifndef AAAC_USE_HINT
#define AAAC_USE_HINT 1
#endif
__device__ __forceinline__ uint32_t interval_hint(const FitTables& S, uint64_t pq) {
#if !AAAC_USE_HINT
    return kNoHint;
#endif
    float P, Q;
    unpack2(pq, P, Q);
    return (S.no_dup && P == P) ? (__float_as_uint(P) & kIdxMask) + (__float_as_uint(Q) & kIdxMask) : kNoHint;
}
struct Exact8 { int J[8]; double emin; int sigma; int tie; };

// Double-precision decision (Eq. 8 as a plain double-precision loop states it, lanes of a group
// combined by a shuffle tree) for the groups whose lanes pass need != 0; every lane of the warp
// calls.  The interval of every weight is found by binary search of the breakpoint list.
template <int LPG>
__device__ __noinline__ Exact8 exact_groups(const FitTables* S, Row8 r, int need) {
    Exact8 out;
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
            const double2 pq = S->PQ[J];
            const double xd = (double)r.x[j], id = (double)r.I[j];
            const double d0 = __dsub_rn(xd, pq.x), d1 = __dsub_rn(xd, pq.y);
            e0 = __dadd_rn(e0, __dmul_rn(id, __dmul_rn(d0, d0)));
            e1 = __dadd_rn(e1, __dmul_rn(id, __dmul_rn(d1, d1)));
        }
        out.J[j] = J;
    }
#pragma unroll
    for (int s = LPG / 2; s; s >>= 1) {
        e0 = __dadd_rn(e0, __shfl_xor_sync(0xFFFFFFFFu, e0, s));
        e1 = __dadd_rn(e1, __shfl_xor_sync(0xFFFFFFFFu, e1, s));
    }
    out.sigma = e1 < e0;
    out.tie = e0 == e1;
    out.emin = out.sigma ? e1 : e0;
    return out;
}

}  // namespace aaac
