// The fit rounds (Algorithm 1 lines 6-16).  With n_inner = 1 a round is the assignment step
// (Eq. 8) and the activation-weighted centroid update (Eq. 11) in a single pass over W, and all
// rounds of a layer run in ONE persistent kernel (one block per SM, cooperative launch): after
// its pass every block adds its sums, as 96-bit fixed-point integers, into 65 global accumulators;
// every 64-bit accumulator word also counts, in its upper 16 bits, the blocks that have added to
// it, so a block knows that a total is complete by reading the total itself -- no separate
// barrier, no fence between the sums and an arrival counter -- and every block ends up with the
// same new tables without a relaunch (integer addition does not depend on the order in which the
// blocks arrive, so the result is bitwise reproducible).  The wait for the totals is bounded: if
// it runs out, the kernel sets AAAC_DEV_TIMEOUT in the device status word and returns.
// With n_inner > 1 the assignment pass (which is also the first inner iteration) stores the
// selection bits, one word per row and 256-column slab, and the remaining n_inner - 1 inner
// iterations are passes of a second instance of the kernel that reads those bits instead of
// forming the two errors; both instances share everything else.  The tables are put in
// ascending order after every pass: in one dimension a centroid update keeps an ascending table
// ascending (ties aside), and the cells depend on the entries' values only, so this equals
// sorting after the last inner iteration.
//
// Per weight the kernel needs (a) the interval J of the merged breakpoint list of both tables
// that holds w~ = fl32(w * r) (Eq. 2) -- J fixes the nearest entry of T0 and of T1 (Eq. 4) --
// (b) its two weighted squared errors, and (c) one accumulation into the centroid sums of cell
// (sigma, J).
//
// (a) Interval.  NB uniform bins on (-8, 8) (512 of width 1/32 here; the pack pass, which has no
//     bins to hold, uses 1024 of width 1/64): with s = NB / 16 the mantissa of
//     fl32(s x + NB / 2 + 1.5 * 2^(23-k)) holds (s x + NB / 2) * 2^k rounded to an integer; masked,
//     it is the byte offset bin * 2^k of the bin's table entry (2^k = bytes per bin over all
//     copies), bin = floor of s x + NB / 2 after rounding to a multiple of 2^-k.
//     A table gives per bin {J_low, thr}: J_low breakpoints lie
//     below the bin, thr is the one breakpoint inside it (+inf if none), J = J_low + (x > thr).
//     Breakpoints are the rounded-down FP32 midpoints, for which x > thr <=> x > midpoint, so J
//     is exact.  A bin that holds two or more breakpoints points at a poisoned slot (J = 31)
//     whose entries are NaN: the group falls through to the exact path below, which searches J
//     directly.  (Fitted tables keep their merged breakpoints apart -- the two codebooks
//     specialise -- so such bins are rare outside degenerate starts.)
// (b) Selection.  A second table gives {P, Q}: the FP32 roundings of the nearest entries of T0
//     and T1 on interval J, moved by at most 8 units in the last place so that the low 4 mantissa
//     bits equal the entry's index (so the
//     same 8 bytes also say which cell the weight falls into).  u_r = x - T_r,
//     E_r = sum_k I_k u_r^2 (Eq. 8), summed per lane and over the lanes of the group by shuffles;
//     sigma = [E1 < E0].
//     Rounding: the constants differ from the entries by at most eta = 17 * 2^-24 max|T|, so
//     |E_r - E_r,exact| <= 2^-24 * 16 E_r + 2 eta sum I |u_r| and
//     sum I |u_r| <= sqrt(sum I * E_r).  Groups with
//     |E0 - E1| <= 2^-24 (16 (E0 + E1) + 2.83 * 17 max|T| sqrt(sum I (E0 + E1))) (and NaN) are
//     re-evaluated in double with the exact entries, so sigma is the double-precision decision
//     (the kernel tests against the slightly larger bound that sqrt(a b) <= a / 16 + 4 b gives,
//     which needs one multiply-add per group).  The two errors are carried as one packed
//     FP32 pair per weight (sub / mul / fma.f32x2).
// (c) Centroid sums, centred.  Lane-private shared-memory bins [sigma][entry] hold
//     (sum I (x - c), sum I) with c the constant of (b) for the entry the weight is assigned to,
//     so the new entry is c + sum I (x - c) / sum I.  The residual sums are small and of mixed
//     sign, which keeps the FP32 accumulation error some 20 times below that of sum I x.  Within
//     a block: no atomics, fixed order.  Across blocks: integer atomics (see above).  After the
//     barrier the centroids are formed (entries of empty cells keep their value) and
//     sorted; block 0 stores the Eq. 8 objective of the round (sum over groups of the smaller
//     error) and, after the last round, the tables.
//
// Tables in shared memory are replicated against bank conflicts: the per-bin table and the
// {P, Q} table 16 times (lane l uses copy l mod 16, so the 16 lanes that share a wavefront of an
// 8-byte load never collide; a bin's entry holds the address of its lower interval's {P, Q} entry
// in the same copy, and a weight above the bin's breakpoint adds the distance to the next
// interval's entry), the bins once per lane.
//
// Thread mapping.  A block of NW warps works on items of 4 NW rows x 256 columns, dealt to
// blocks as contiguous ranges (slab-major), so every sum has a fixed order and results are
// bitwise reproducible.  A warp takes 4 rows; each lane 8 adjacent columns (one 128-bit load
// per row), so its eight importances stay in registers.  A group is 2 lanes (g = 16) or 16
// lanes (g = 128).  A row's registers are refilled from the next item right after the row is unpacked.
#include <type_traits>

#include "lookup.cuh"

namespace aaac {

namespace {

struct FitParams {
    const uint16_t* W;
    int64_t N, K, ldw;
    const uint8_t* scales;        // NVFP4 scale bytes
    const float* rinv;            // INT4 reciprocal scales
    const float* I;
    Ctrl* ctrl;
    unsigned long long* acc;      // [3][kUsed][3] words, 128 bytes apart: fixed-point sums over the blocks, one buffer per pass in rotation
    double* err_trace;            // [n_rounds] or null
    float* T01_out;               // [2][16] or null: the tables after the launch's last pass, as FP32
    uint32_t* dev_status;         // or null
    uint32_t* sigw;               // [N][slabs]: selection bits of a row's 256-column slab, bit = lane (n_inner > 1)
    int n_rounds;                 // passes over W in this launch
    int trace_base;               // err_trace index of this launch's first assignment pass
    unsigned bar_base;            // passes of the layer's earlier launches (the sum buffers rotate per pass)
    unsigned arrivals;            // blocks whose sums a total must hold before it is read (the grid size)
    unsigned spin_limit;          // polls of a total before the wait is given up
    int items, per_block, nrb;    // (4 NW)-row x 256-column items, items per block, row blocks per slab
    int tail_item0, tail_quarters;   // items from tail_item0 on are dealt out a quarter (one row per warp) per block
};

constexpr uint32_t kLut1At = 65536;                    // shared address of the bin table (see fit_rounds_body)
constexpr int kMaxFitBlocks = 1024;                   // grid limit: block sums are added as 32-bit limbs, the arrivals counted in 16 bits
constexpr int kLimbs = 3;                             // a sum is a 96-bit two's-complement fixed-point number
constexpr unsigned kDefaultSpinLimit = 1u << 23;      // polls of >= 32 ns each: several seconds
constexpr int kAccStride = 16;                        // accumulator words lie 128 bytes apart: one cache line each, so that the
                                                      // blocks' atomics on different sums do not queue behind one another
constexpr int kAccBuffer = kUsed * kLimbs * kAccStride;   // 64-bit words of one pass's buffer
constexpr int kCountShift = 48;                       // an accumulator word: limb sum below, arrivals above
constexpr unsigned long long kLimbMask = (1ull << kCountShift) - 1ull;
constexpr unsigned long long kOneArrival = 1ull << kCountShift;
constexpr long long kTopBias = 1ll << 31;             // added to the (signed) top limb so that every block adds a non-negative number

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// process-wide knobs of the wait (aaac_debug_fit_wait): extra arrivals a total must show before it is
// taken (0 in normal use; 1 makes every wait run out) and the poll limit
int g_extra_arrivals = 0;
unsigned g_spin_limit = kDefaultSpinLimit;

// Near-tie groups are not decided inside the row pipeline: their lanes send the row's centred
// terms to a spare bin slot that nobody reads, the group goes on a short per-warp list, and
// resolve_deferred (after the pass's items, or when the list fills up) decides it in double and
// adds its weights to the bins.  That keeps the hot loop free of the slow path, whose latency every
// pass would otherwise pay on the warp that drew the most near-ties.
constexpr int kDeferCap = 96;                         // list entries per warp: {row, first column of the group}
constexpr int kBinSlots = kCells + 1;                 // [sigma][entry] and the spare slot
constexpr int kSpareSlot = kCells;

__device__ __forceinline__ void sts_u2(uint32_t addr, uint32_t a, uint32_t b) {
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" :: "r"(addr), "r"(a), "r"(b) : "memory");
}

// A launch runs passes of one kind.  kRounds: assignment passes, each also the (only) inner
// iteration of its round -- the n_inner = 1 procedure, all rounds of a layer in one launch.
// kAssignKeep: the same pass, which also stores the selection bits.  kInner: further inner
// iterations with the stored selection.  With n_inner > 1 a round is one kAssignKeep launch of a
// single pass followed by one kInner launch of n_inner - 1 passes.
enum PassKind { kRounds = 0, kAssignKeep = 1, kInner = 2 };

// Decides the listed selection groups in double (Eq. 8: each lane adds its weights' terms in index
// order, the lanes of the group are combined pairwise; a tie goes to table 0) and adds every weight
// to the calling lane's bins under the chosen table, with the arithmetic of the row pipeline
// (centred term I (x - c), c the chosen entry's centre constant).  Every lane of the warp calls;
// returns the sum of the groups' smaller errors in lane 0 (0 elsewhere).
struct DeferArgs {                // what the routine needs of the layer (passed by value: the kernel's
    const uint16_t* W;            // parameters themselves stay where they are)
    int64_t K, ldw;
    const uint8_t* scales;
    const float* rinv;
    const float* I;
    uint32_t* sigw;
};
template <int MODE, int SEL, int KIND>
__device__ __noinline__ double resolve_deferred(const FitTables* S, const DeferArgs p, uint32_t list_addr, int count,
                                                uint32_t bins_lane, int lane) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;      // scale group
    constexpr int WPL = SEL >= 32 ? SEL / 32 : 1;        // weights per lane
    constexpr int ACTIVE = SEL / WPL;                    // lanes that hold weights of the group (32 or 16)
    constexpr int LPG = SEL / 8;                         // lanes of the group in the row pipeline
    const int K = (int)p.K, Gr = K / G, slabs = (K + 255) >> 8;
    double esum = 0.0;
    for (int e = 0; e < count; ++e) {
        uint32_t urow, ucol;
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(urow), "=r"(ucol) : "r"(list_addr + (uint32_t)e * 8u));
        const int row = (int)urow, cg = (int)ucol;
        float xs[WPL], Is[WPL];
        int Js[WPL];
        double e0 = 0.0, e1 = 0.0;
        if (lane < ACTIVE) {
#pragma unroll
            for (int t = 0; t < WPL; ++t) {
                const int col = cg + lane * WPL + t;
                const uint32_t wb = p.W[(size_t)row * (size_t)p.ldw + col];
                const size_t gi = (size_t)row * (size_t)Gr + (uint32_t)col / G;
                const float rinv = MODE == AAAC_NVFP4 ? S->rlut[p.scales[gi] & 0x7Fu] : __ldg(p.rinv + gi);
                const float x = __fmul_rn(__uint_as_float(wb << 16), rinv);
                const float iv = __ldg(p.I + col);
                int J = 0;
#pragma unroll
                for (int step = 16; step; step >>= 1)      // number of breakpoints below x (sorted list)
                    if (J + step <= kNBP && S->bp[J + step - 1] < x) J += step;
                const double2 pq = S->PQ[J];
                const double xd = (double)x, id = (double)iv;
                const double d0 = __dsub_rn(xd, pq.x), d1 = __dsub_rn(xd, pq.y);
                e0 = __dadd_rn(e0, __dmul_rn(id, __dmul_rn(d0, d0)));
                e1 = __dadd_rn(e1, __dmul_rn(id, __dmul_rn(d1, d1)));
                xs[t] = x; Is[t] = iv; Js[t] = J;
            }
        }
#pragma unroll
        for (int o = ACTIVE / 2; o; o >>= 1) {
            e0 = __dadd_rn(e0, __shfl_xor_sync(0xFFFFFFFFu, e0, o));
            e1 = __dadd_rn(e1, __shfl_xor_sync(0xFFFFFFFFu, e1, o));
        }
        e0 = __shfl_sync(0xFFFFFFFFu, e0, 0);
        e1 = __shfl_sync(0xFFFFFFFFu, e1, 0);
        const bool sg = e1 < e0;
        if (lane < ACTIVE) {
#pragma unroll
            for (int t = 0; t < WPL; ++t) {
                const float2 c2 = S->pq32[Js[t]];
                const float c = sg ? c2.y : c2.x;
                const uint32_t a = bins_lane + ((sg ? (uint32_t)kM : 0u) + (__float_as_uint(c) & kIdxMask)) * kSlotBytes;
                float2 b = lds_bin(a);
                b.x += __fmul_rn(Is[t], __fsub_rn(xs[t], c));
                b.y += Is[t];
                sts_bin(a, b);
            }
        }
        if (lane == 0) {
            esum += sg ? e1 : e0;
            if (KIND == kAssignKeep) {
                // the stored selection bits of the row's slab: bit = lane of the row pipeline
                const uint32_t first = ((uint32_t)cg & 255u) >> 3;
                const uint32_t mask = (LPG >= 32 ? 0xFFFFFFFFu : ((1u << LPG) - 1u)) << first;
                uint32_t* wp = p.sigw + (size_t)row * (size_t)slabs + (cg >> 8);
                const uint32_t old = *wp;
                *wp = sg ? (old | mask) : (old & ~mask);
            }
        }
    }
    return esum;
}

// SEL is the selection group size S (Sec. 3.1): the weights that share one codebook choice; the
// scale group g is fixed by the format.
// The passes of one layer, run by the nblk blocks bid = 0 .. nblk - 1 (a whole grid, or the part
// of a grid that a batch of layers gives to this layer).
template <int MODE, int SEL, int NW, int REP, int KIND>
__device__ __forceinline__ void fit_rounds_body(const FitParams& p, const unsigned bid, const unsigned nblk) {
    constexpr int NB = AAAC_FIT_BINS;
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;      // scale group
    constexpr int LPG = SEL / 8;                         // lanes per selection group
    constexpr int R = kRowsPerWarp;
    constexpr int kRowsPerItem = R * NW;
    constexpr int NT = NW * 32;
    constexpr int kLut1Bytes = REP * NB * 8;
    constexpr int kBinBytes = kBinSlots * kSlotBytes;        // per warp
    static_assert(kLut1Bytes >= NW * kPartStride * 8, "the per-warp partials reuse the first table's space");
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ FitTables S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // 32-bit shared addresses.  The bin table sits at a shared address that is a multiple of its own
    // span (64 KB), so that a lookup's address -- bin bits, the lane's copy and the table base -- is one
    // three-input logic instruction; the bins of the first warps fill the space below it, the other
    // warps' bins, the {P, Q} table and the near-tie lists follow it.  Slot offsets carry the address of
    // this lane's column of the {P, Q} table, so a lookup there needs no further arithmetic.
    static_assert(kLut1Bytes == (int)kLut1At, "the bin table spans exactly the alignment of its address");
    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(dyn);
    uint32_t dyn_size;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_size));
    const uint32_t gap = kLut1At - sm_base;                                            // bytes of the dynamic region below the table
    const int n_low = min(NW, (int)(gap / (uint32_t)kBinBytes));                       // warps whose bins lie below the table
    const uint32_t hi_base = kLut1At + kLut1Bytes;
    const uint32_t lut2_addr = hi_base + (uint32_t)(NW - n_low) * kBinBytes;           // the {P, Q} table
    const uint32_t lists_at = lut2_addr + kLut2Bytes;
    if (sm_base > kLut1At || lists_at + NW * (kDeferCap * 8) > sm_base + dyn_size) {
        // the layout does not fit the shared memory this launch was given (the same for every block, so
        // all of them leave before any of them waits): reported like a wait that ran out -- no valid result
        if (bid == 0 && threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, AAAC_DEV_TIMEOUT);
        return;
    }
    unsigned char* const lut1_mem = dyn + gap;
    unsigned char* const lut2_mem = dyn + (lut2_addr - sm_base);
    const uint32_t lut1_or = kLut1At | ((lane & (REP - 1)) * 8);                        // table base | this lane's copy of a bin's entry; | bin * REP * 8
    const uint32_t bins_warp = warp < n_low ? sm_base + warp * kBinBytes : hi_base + (uint32_t)(warp - n_low) * kBinBytes;
    const uint32_t bins_lane = bins_warp + lane * 8;                                   // + cell * 256
    const uint32_t spare_lane = bins_lane + kSpareSlot * kSlotBytes;                   // sink of the near-tie groups' rows
    const uint32_t list_addr = lists_at + warp * (kDeferCap * 8);
    double* wsum = reinterpret_cast<double*>(lut1_mem);    // [NW][kPartStride], over the first table

    // 32-bit index arithmetic throughout (N, K < 2^31); only the final element offsets are 64-bit
    const int N = (int)p.N, K = (int)p.K;
    const int Gr = K / G;
    const int slabs = (K + 255) >> 8;
    // A block takes a contiguous range of whole items; what does not divide evenly (the items from
    // tail_item0 on) is dealt out one quarter item -- one row per warp -- per block, so that the
    // busiest block has at most a quarter item more than the others.
    const int it0 = (int)bid * p.per_block;
    const int it1 = min(p.tail_item0, it0 + p.per_block);
    const bool has_tail = (int)bid < p.tail_quarters;
    const int tail_item = p.tail_item0 + ((int)bid >> 2), tail_u = (int)bid & 3;
    static_assert(R == 4, "a tail quarter is one of the four rows of a warp");

    if (tid < 2 * kM) S.Td[tid] = p.ctrl->T[tid];
    if (MODE == AAAC_NVFP4 && tid >= 64 && tid < 192) {
        const int c = tid - 64;
        const float sv = __fmul_rn(e4m3_value((uint32_t)c), p.ctrl->s_t);
        S.rlut[c] = c ? __frcp_rn(sv) : 0.f;
    }
    __syncthreads();

    // Fixed-point scale of the sums over the blocks.  Every sum of a pass is bounded by
    // B = 256 N K max_k I_k (|w~ - c| < 16), so with 2^e > B the value v 2^(94 - e) fits 96 bits; what
    // is dropped lies 2^-86 below B.  Integer addition is order-independent, so the totals do not
    // depend on the order in which the blocks arrive (max is order-independent too).
    {
        float mx = 0.f;
        for (int k = tid; k < K; k += NT) mx = fmaxf(mx, fabsf(__ldg(p.I + k)));
#pragma unroll
        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        float* red = reinterpret_cast<float*>(lut1_mem);
        if (lane == 0) red[warp] = mx;
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < NW; ++w) mx = fmaxf(mx, red[w]);
            const double B = 256.0 * (double)N * (double)K * (double)mx;
            int e = 0;
            if (B > 0.0 && B < 1e300) e = ilogb(B) + 1;
            S.fix_scale = scalbn(1.0, 94 - e);
            S.fix_unscale = scalbn(1.0, e - 94);
        }
        __syncthreads();
    }

    // bin arithmetic: the masked mantissa of fl32(kBinsPerUnit x + kMagic) is bin * (REP * 8)
    constexpr float kBinsPerUnit = (float)(NB / 16);
    constexpr float kMagic = (float)(NB / 2) + 1.5f * (float)(1 << 23) / (float)(REP * 8);
    constexpr uint32_t kBinMask = (uint32_t)(NB - 1) * (REP * 8);

    for (int b = 0; b < kCells; ++b) sts_bin(bins_lane + b * kSlotBytes, make_float2(0.f, 0.f));
  for (int round = 0; round < p.n_rounds; ++round) {
    const unsigned pass_no = p.bar_base + (unsigned)round;
    // block 0 clears the buffer of the next pass: it was the buffer of two passes ago, and every block
    // finished reading it before it added to the previous pass's buffer, whose totals block 0 has seen
    static_assert(NT >= 256 + kUsed * kLimbs, "threads 256.. of block 0 clear the next buffer");
    if (bid == 0 && tid >= 256 && tid < 256 + kUsed * kLimbs) {
        p.acc[(size_t)((pass_no + 1u) % 3u) * kAccBuffer + (size_t)(tid - 256) * kAccStride] = 0ull;
        __threadfence();
    }
    build_tables<MODE, NW, REP, NB>(S, lut1_mem, lut2_mem);
    // near-tie bound: sqrt(a b) <= (kappa a + b / kappa) / 2, so the bound of the header comment is at
    // most g1 * (E0 + E1) + g2 * sum I, with kappa = 1/8 (about the usual |w~ - entry|)
    const float g1 = 0x1p-24f * __fmaf_ru(S.tmax283, 4.f, 16.f), g2 = 0x1p-24f * __fmul_ru(S.tmax283, 0.0625f);
    double Eacc = 0.0;

   auto pass = [&](auto inner_tag) {
    constexpr bool INNER = decltype(inner_tag)::value;
    constexpr bool keep_sigma = KIND == kAssignKeep;
    // Row registers of the item being processed; a row's registers are refilled with the same row
    // of the next item as soon as the row has been unpacked, so the load has about an item's time
    // to arrive and no second buffer is needed.
    uint4 v[R];
    uint32_t sc[R];           // NVFP4: scale byte; INT4: bits of the reciprocal scale
    uint32_t sgw[R];          // inner iteration: the row's stored selection bits
    // (An unguarded form with clamped indices was measured too: faster for some instantiations, slower
    // for others, depending on what else the kernel held; the guarded form is the one kept.)
    auto load_row = [&](int u, int slab, int rb) {
        const int col0 = slab * 256 + lane * 8;
        const int row = rb * kRowsPerItem + warp * R + u;
        v[u] = make_uint4(0, 0, 0, 0);
        sc[u] = 0u;
        if (INNER) sgw[u] = 0u;
        if (col0 < K && row < N) {
            // element offsets fit 32 bits (the entry points refuse layers of 2^32 elements and more)
            v[u] = __ldcs(reinterpret_cast<const uint4*>(p.W + ((unsigned)row * (unsigned)p.ldw + (unsigned)col0)));
            const unsigned gi = (unsigned)row * (unsigned)Gr + (unsigned)col0 / G;
            if (MODE == AAAC_NVFP4) sc[u] = p.scales[gi];          // masked at use: nothing waits on the load here
            else sc[u] = __float_as_uint(__ldg(p.rinv + gi));
            if (INNER) sgw[u] = __ldcg(p.sigw + (size_t)row * (size_t)slabs + slab);
        }
    };

    int cur_slab = -1;
    int ndefer = 0;           // groups on the warp's list (the same in every lane)
    uint64_t II[8];           // {I, I} of the lane's eight columns
    float isum = 0.f;         // g2 * sum of I over the lane's group (rounded up a little)
    bool col_ok = false;
#pragma unroll
    for (int j = 0; j < 8; ++j) II[j] = 0ull;

    // (slab, row block) of the current item and of the one being loaded
    const int n_main = max(it1 - it0, 0), n_items = n_main + (has_tail ? 1 : 0);
    const int first = n_main > 0 ? it0 : tail_item;
    int slab = first / p.nrb, rb = first - slab * p.nrb;
    int nslab = slab, nrb = rb;
    if (n_items > 0) {
#pragma unroll
        for (int u = 0; u < R; ++u) load_row(u, slab, rb);
    }
    for (int i = 0; i < n_items; ++i) {
        slab = nslab;
        rb = nrb;
        if (i + 1 < n_main) {
            if (++nrb == p.nrb) { nrb = 0; ++nslab; }
        } else {                                           // the tail item comes next (if any)
            nslab = tail_item / p.nrb;
            nrb = tail_item - nslab * p.nrb;
        }
        // After the last item nothing follows: its own rows are fetched once more (in bounds, unused), so
        // that the loads of the next item's rows stand in the row pipeline without a branch around them
        // (with one, the compiler kept them from moving: 799 -> 835 Gweights/s on the benchmark layers).
        if (i + 1 >= n_items) { nslab = slab; nrb = rb; }
        const bool whole = i < n_main;                     // else: row tail_u of every warp only

        if (slab != cur_slab) {
            cur_slab = slab;
            const int col0 = slab * 256 + lane * 8;
            col_ok = col0 < K;
            isum = 0.f;
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
        const int row0 = rb * kRowsPerItem + warp * R;
        const int nrows = min(R, N - row0);                // rows of this warp inside the layer (may be <= 0)

        // The rows of the item go through three stages, written out in the order in which the
        // shared-memory operations are to be issued, so that the read-modify-write chain on the
        // bins of one row runs while the table lookups of the next row are in flight:
        //   L1(u): w~ and the loads of {J_low, thr};   L2(u): slot and the loads of {P, Q};
        //   M(u):  errors, sigma, the centred terms and bin addresses;   B(u): bins += terms.
        float eitem = 0.f;                                 // objective of this item's groups led by this lane
        float x[8];                                        // w~ of the row in L1..M
        uint2 e1v[8];                                      // {address of the lower interval's {P, Q} entry, thr}
        uint64_t pq[8];                                    // {P, Q}, packed
        float mt[2][8];                                    // chosen centred term I (x - c) of the rows in B / M
        uint32_t ba[2][8];                                 // its bin address
        bool sg_row = false;                               // inner iteration: this lane's stored selection bit
        auto L1 = [&](int u) {
            if (INNER) sg_row = (sgw[u] >> lane) & 1u;
            const float rinv = MODE == AAAC_NVFP4 ? S.rlut[sc[u] & 0x7Fu] : __uint_as_float(sc[u]);
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                x[j] = __fmul_rn((j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]), rinv);
                // (bin bits | lane's copy) is one three-input logic instruction, and the table's base, the
                // same for every lane, can ride in the load's address: no add per weight
                e1v[j] = lds_table_u2(((uint32_t)__float_as_int(__fmaf_rn(x[j], kBinsPerUnit, kMagic)) & kBinMask) | lut1_or);
            }
        };
        // same, then refill the row's registers from the next item
        auto L1n = [&](int u) {
            L1(u);
            load_row(u, nslab, nrb);
        };
        auto L2 = [&]() {
#pragma unroll
            for (int j = 0; j < 8; ++j) pq[j] = lds_table_b64(above_addr(e1v[j].x, x[j], e1v[j].y));
        };
        auto M = [&](int row, float (&mt_o)[8], uint32_t (&ba_o)[8]) {
            if constexpr (INNER) {
                // selection frozen: the centred term under the stored table only.  A poisoned
                // slot shows as NaN; those lanes search their intervals directly.
                const bool sg = sg_row;
                float c[8], chk = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float cP, cQ;
                    unpack2(pq[j], cP, cQ);
                    c[j] = sg ? cQ : cP;
                    mt_o[j] = __fmul_rn(lo2(II[j]), __fsub_rn(x[j], c[j]));
                    chk += mt_o[j];
                }
                const bool bad = !(chk == chk);
                if (__any_sync(0xFFFFFFFFu, bad)) {
                    Row8 r;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { r.x[j] = x[j]; r.I[j] = lo2(II[j]); r.hint[j] = kNoHint; }
                    const Exact8 ex = exact_groups<LPG>(&S, r, (int)bad);
                    if (bad) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float cP, cQ;
                            unpack2(lds_table_b64(pq_entry_addr(lut2_addr, ex.J[j], lane)), cP, cQ);
                            c[j] = sg ? cQ : cP;
                            mt_o[j] = __fmul_rn(lo2(II[j]), __fsub_rn(x[j], c[j]));
                        }
                    }
                }
                const uint32_t base = bins_lane + (sg ? kM * kSlotBytes : 0);
#pragma unroll
                for (int j = 0; j < 8; ++j) ba_o[j] = base + (__float_as_uint(c[j]) & kIdxMask) * kSlotBytes;
                return;
            }
            uint64_t m[8];                                 // {I (x - P), I (x - Q)}
            uint64_t e01 = 0ull;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint64_t u01 = diff2(x[j], pq[j]);
                m[j] = mul2(II[j], u01);
                e01 = fma2(m[j], u01, e01);
            }
            float e0 = lo2(e01), e1 = hi2(e01);
#pragma unroll
            for (int s = LPG / 2; s; s >>= 1) {
                e0 += __shfl_xor_sync(0xFFFFFFFFu, e0, s);
                e1 += __shfl_xor_sync(0xFFFFFFFFu, e1, s);
            }
            const float es = e0 + e1;
            const float tau = __fmaf_ru(es, g1, isum);
            // lanes past K carry I = 0 and w~ = 0; they need the exact path only if their slot is
            // poisoned (NaN), so that no NaN reaches a bin
            const bool near = !(fabsf(e1 - e0) > tau) && (col_ok || !(es == es));
            const bool sg = e1 < e0;
            float emin = sg ? e1 : e0;
            uint32_t base = bins_lane + (sg ? kM * kSlotBytes : 0), idx_mask = kIdxMask;
            if (__any_sync(0xFFFFFFFFu, near)) {
                // near-ties and poisoned slots (rare): the group goes on the warp's list, to be decided
                // in double by resolve_deferred; its lanes send this row's terms to the spare slot
                const bool lead = near && col_ok && (lane % LPG) == 0;
                const unsigned lm = __ballot_sync(0xFFFFFFFFu, lead);
                if (lead) sts_u2(list_addr + (uint32_t)(ndefer + __popc(lm & ((1u << lane) - 1u))) * 8u, (uint32_t)row,
                                 (uint32_t)(slab * 256 + lane * 8));
                ndefer += __popc(lm);
                if (near) { emin = 0.f; base = spare_lane; idx_mask = 0u; }
            }
            if (col_ok && (lane % LPG) == 0) eitem += emin;
            if (keep_sigma) {
                const unsigned bits = __ballot_sync(0xFFFFFFFFu, sg);        // (the bits of listed groups are set when they are decided)
                if (lane == 0) p.sigw[(size_t)row * (size_t)slabs + slab] = bits;
            }
            // cell = entry index (low bits of the centre constant) under the chosen table
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float m0, m1, cP, cQ;
                unpack2(m[j], m0, m1);
                unpack2(pq[j], cP, cQ);
                mt_o[j] = sg ? m1 : m0;
                ba_o[j] = base + (__float_as_uint(sg ? cQ : cP) & idx_mask) * kSlotBytes;
            }
        };
        auto B = [&](const float (&mt_i)[8], const uint32_t (&ba_i)[8], int j0, int j1) {
#pragma unroll
            for (int j = j0; j < j1; ++j) {
                float2 a = lds_bin(ba_i[j]);
                a.x += mt_i[j];
                a.y += lo2(II[j]);
                sts_bin(ba_i[j], a);
            }
        };

        if (nrows == R && whole) {
            // full item: L1(0) L2(0) M(0) | L1(1) B(0)[0..1] L2(1) B(0)[2..7] M(1) | ... | B(R-1)
            // (where the second lookups cut into the previous row's bin updates was chosen by measurement: 2 + 6)
            L1n(0);
            L2();
            M(row0, mt[0], ba[0]);
#pragma unroll
            for (int u = 1; u < R; ++u) {
                const int prev = (u - 1) & 1, cur = u & 1;
                L1n(u);
                B(mt[prev], ba[prev], 0, 2);
                L2();
                B(mt[prev], ba[prev], 2, 8);
                M(row0 + u, mt[cur], ba[cur]);
            }
            B(mt[(R - 1) & 1], ba[(R - 1) & 1], 0, 8);
        } else {
            // ragged last row block of the layer: row by row, then refill all rows
            uint4 vr[R];
            uint32_t sr[R], gr[R];
#pragma unroll
            for (int t = 0; t < R; ++t) { vr[t] = v[t]; sr[t] = sc[t]; gr[t] = INNER ? sgw[t] : 0u; }
            const int ulo = whole ? 0 : tail_u, uhi = whole ? nrows : min(nrows, tail_u + 1);
            for (int u = ulo; u < uhi; ++u) {
                // (u is uniform over the warp; the stages read row 0 of v[] and sc[])
#pragma unroll
                for (int t = 0; t < R; ++t)
                    if (u == t) { v[0] = vr[t]; sc[0] = sr[t]; if (INNER) sgw[0] = gr[t]; }
                L1(0);
                L2();
                M(row0 + u, mt[0], ba[0]);
                B(mt[0], ba[0], 0, 8);
            }
#pragma unroll
            for (int t = 0; t < R; ++t) load_row(t, nslab, nrb);
        }
        Eacc += (double)eitem;
        if (!INNER && ndefer > kDeferCap - R * (32 / LPG)) {    // the next item could overflow the list
            __syncwarp();
            Eacc += resolve_deferred<MODE, SEL, KIND>(&S, DeferArgs{p.W, p.K, p.ldw, p.scales, p.rinv, p.I, p.sigw}, list_addr, ndefer, bins_lane, lane);
            ndefer = 0;
        }
    }
    if (!INNER && ndefer > 0) {
        __syncwarp();
        Eacc += resolve_deferred<MODE, SEL, KIND>(&S, DeferArgs{p.W, p.K, p.ldw, p.scales, p.rinv, p.I, p.sigw}, list_addr, ndefer, bins_lane, lane);
    }
   };
    pass(std::integral_constant<bool, KIND == kInner>{});

    // ---- block partial: lane c of a warp adds the 32 lane-private values of cell c (in a
    //      rotated, fixed order that avoids bank conflicts); then the warps are added ----
    __syncthreads();                                       // every warp is done with the lookup tables
    {
        // four interleaved chains in double: 32 FP32 values go into 53 bits without rounding unless they
        // are more than 2^24 apart, and then by less than 2^-52 of the sum
        double dx[4] = {0.0, 0.0, 0.0, 0.0}, dy[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float2 a = lds_bin(bins_warp + lane * kSlotBytes + ((i + lane) & 31) * 8);
            dx[i & 3] += (double)a.x;
            dy[i & 3] += (double)a.y;
        }
        wsum[warp * kPartStride + lane] = (dx[0] + dx[1]) + (dx[2] + dx[3]);
        wsum[warp * kPartStride + kCells + lane] = (dy[0] + dy[1]) + (dy[2] + dy[3]);
        // the warp's bins start the next pass at zero (done here, ahead of the wait for the totals)
        __syncwarp();
#pragma unroll 8
        for (int b = 0; b < kCells; ++b) sts_bin(bins_lane + b * kSlotBytes, make_float2(0.f, 0.f));
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) Eacc += __shfl_xor_sync(0xFFFFFFFFu, Eacc, s);
    if (lane == 0) wsum[warp * kPartStride + 2 * kCells] = Eacc;
    __syncthreads();
    // this block's sums go into the pass's buffer as three 32-bit limbs of a 96-bit fixed-point number,
    // each with one arrival in the word's upper bits
    unsigned long long* acc = p.acc + (size_t)(pass_no % 3u) * kAccBuffer + (size_t)tid * (kLimbs * kAccStride);   // this thread's three words
    const unsigned long long want = (unsigned long long)p.arrivals;
    bool ok = true;
    if (tid < kUsed) {
        double ws_[NW];                                     // the warps' sums, added pairwise (a fixed order)
#pragma unroll
        for (int w = 0; w < NW; ++w) ws_[w] = wsum[w * kPartStride + tid];
#pragma unroll
        for (int stride = 1; stride < NW; stride *= 2)
#pragma unroll
            for (int w = 0; w + stride < NW; w += 2 * stride) ws_[w] += ws_[w + stride];
        const double sd = ws_[0] * S.fix_scale;
        const double t2 = floor(sd * 0x1p-64);             // in [-2^30, 2^30)
        const double r = sd - t2 * 0x1p64;                 // exact, in [0, 2^64)
        const double t1 = floor(r * 0x1p-32);
        const double t0 = floor(r - t1 * 0x1p32);
        atomicAdd(acc + 0 * kAccStride, (unsigned long long)t0 + kOneArrival);
        atomicAdd(acc + 1 * kAccStride, (unsigned long long)t1 + kOneArrival);
        atomicAdd(acc + 2 * kAccStride, (unsigned long long)((long long)t2 + kTopBias) + kOneArrival);
    }
    // ---- wait until every block's sums are in, then read the totals.  One thread of the block
    //      polls one word (all blocks add all their words at about the same time; a crowd of
    //      pollers on the accumulators' cache lines would hold the atomics up); after it every
    //      thread checks the arrival counts of its own words and waits on if they are short ----
#ifndef AAAC_FIT_POLL_ALL
#define AAAC_FIT_POLL_ALL 0
#endif
#if !AAAC_FIT_POLL_ALL
    if (tid == kUsed - 1) {
        for (unsigned spins = 0;; ++spins) {
            if ((ld_relaxed_u64(acc) >> kCountShift) >= want) break;
            if (spins >= p.spin_limit || ld_relaxed_u32(&p.ctrl->abort)) { ok = false; break; }
            __nanosleep(32);
        }
    }
    __syncthreads();
#endif
    if (tid < kUsed) {
        unsigned long long w0, w1, w2;
        for (unsigned spins = 0;; ++spins) {
            w0 = ld_relaxed_u64(acc + 0 * kAccStride);
            w1 = ld_relaxed_u64(acc + 1 * kAccStride);
            w2 = ld_relaxed_u64(acc + 2 * kAccStride);
            if ((w0 >> kCountShift) >= want && (w1 >> kCountShift) >= want && (w2 >> kCountShift) >= want) break;
            if (spins >= p.spin_limit || ld_relaxed_u32(&p.ctrl->abort)) { ok = false; break; }
            __nanosleep(64);
        }
        const long long l2 = (long long)(w2 & kLimbMask) - (long long)nblk * kTopBias;
        __int128 v = ((__int128)l2 << 64) + ((__int128)(w1 & kLimbMask) << 32) + (__int128)(w0 & kLimbMask);
        const bool neg = v < 0;
        if (neg) v = -v;
        const double mag = (double)(unsigned long long)(v >> 64) * 0x1p64 + (double)(unsigned long long)v;
        S.tot[tid] = (neg ? -mag : mag) * S.fix_unscale;
    }
    if (!__syncthreads_and(ok)) {
        // a wait ran out (here or in another block): tell the others, report, leave
        if (tid == 0) {
            atomicExch(&p.ctrl->abort, 1u);
            if (p.dev_status) atomicOr(p.dev_status, AAAC_DEV_TIMEOUT);
        }
        return;
    }
    if (tid < 2 * kM) {
        // cells of duplicate entries are empty: they keep their value
        const double sx = S.tot[tid], wt = S.tot[kCells + tid];
        S.tot[2 * kCells + 1 + tid] = (wt > 0.0) ? (double)S.centre[tid] + __ddiv_rn(sx, wt) : S.Td[tid];
    }
    __syncthreads();
    if (tid < 2 * kM) {
        // ascending order within the table by rank (ties by index)
        const double* tn = S.tot + 2 * kCells + 1 + (tid & 16);
        const double t = tn[tid & 15];
        int rank = 0;
#pragma unroll 1
        for (int i = 0; i < kM; ++i) rank += (tn[i] < t) || (tn[i] == t && i < (tid & 15));
        S.Td[(tid & 16) + rank] = t;
    }
    // the trace holds the Eq. 8 objective of each assignment step
    if (KIND != kInner && bid == 0 && tid == 0 && p.err_trace)
        p.err_trace[p.trace_base + round] = S.tot[2 * kCells];
    __syncthreads();
  }
    if (bid == 0 && tid < 2 * kM) {
        p.ctrl->T[tid] = S.Td[tid];
        if (p.T01_out) p.T01_out[tid] = (float)S.Td[tid];
    }
}

template <int MODE, int SEL, int NW, int REP, int KIND>
__global__ void __launch_bounds__(NW * 32, 1) fit_rounds_kernel(const FitParams p) {
    fit_rounds_body<MODE, SEL, NW, REP, KIND>(p, blockIdx.x, gridDim.x);
}

// Several layers in one launch (the paper processes layers independently, Sec. 3.3): the grid is
// cut into consecutive ranges of blocks, one per layer, and every range runs that layer's rounds
// by itself -- its blocks wait only for each other, on the layer's own accumulators -- so the
// per-round fixed cost (sums across blocks, new tables, table building) is paid once for the
// whole batch instead of once per layer, and small layers no longer leave most of the GPU idle.
// The parameters of every layer stay kernel arguments (one copy of the code per slot).
constexpr int kMaxBatch = 8;
struct FitBatch {
    FitParams L[kMaxBatch];
    unsigned first[kMaxBatch + 1];    // first block of every layer; first[n..] = grid size
};

template <int MODE, int SEL, int NW, int REP>
__global__ void __launch_bounds__(NW * 32, 1) fit_batch_kernel(const FitBatch b) {
    const unsigned bx = blockIdx.x;
#define AAAC_BATCH_SLOT(i)                                                                              \
    if (bx < b.first[i + 1]) {                                                                           \
        fit_rounds_body<MODE, SEL, NW, REP, kRounds>(b.L[i], bx - b.first[i], b.first[i + 1] - b.first[i]); \
        return;                                                                                          \
    }
    AAAC_BATCH_SLOT(0) AAAC_BATCH_SLOT(1) AAAC_BATCH_SLOT(2) AAAC_BATCH_SLOT(3)
    AAAC_BATCH_SLOT(4) AAAC_BATCH_SLOT(5) AAAC_BATCH_SLOT(6) AAAC_BATCH_SLOT(7)
#undef AAAC_BATCH_SLOT
}

__global__ void export_tables_kernel(const Ctrl* ctrl, float* T01) {
    if (threadIdx.x < 2 * kM) T01[threadIdx.x] = (float)ctrl->T[threadIdx.x];
}

// The fit kernels place their tables at fixed shared addresses and take all the shared memory a block
// may have beyond their static part (one block per SM either way); the kernel checks that its layout fits.
cudaError_t fit_dynamic_smem(const void* kern, size_t* bytes) {
    cudaFuncAttributes a;
    cudaError_t e = cudaFuncGetAttributes(&a, kern);
    if (e != cudaSuccess) return e;
    int dev = 0, optin = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
    if ((size_t)optin <= a.sharedSizeBytes) return cudaErrorInvalidValue;
    *bytes = (size_t)optin - a.sharedSizeBytes;
    return cudaSuccess;
}

template <int MODE, int SEL, int NW, int REP, int KIND>
cudaError_t launch_variant(FitParams& p, unsigned grid, cudaStream_t st) {
    auto kern = fit_rounds_kernel<MODE, SEL, NW, REP, KIND>;
    size_t smem = 0;
    cudaError_t e = fit_dynamic_smem(reinterpret_cast<const void*>(kern), &smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    void* args[] = {&p};
    note_launch();
    // cooperative: every block is resident, which the grid-wide barrier relies on
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kern), dim3(grid), dim3(NW * 32), args, smem, st);
}

}  // namespace

// Deals a layer's items to `blocks` blocks: whole items in contiguous ranges plus, where that is
// shorter for the busiest block, a tail dealt out one row per warp (a quarter item) per block.
// Returns the number of blocks actually used.
static int64_t plan_layer(FitParams& p, int64_t N, int64_t K, int64_t blocks) {
    const int64_t slabs = (K + 255) / 256;
    constexpr int kRowsPerItem = kRowsPerWarp * AAAC_FIT_WARPS;
    const int64_t nrb = (N + kRowsPerItem - 1) / kRowsPerItem, items = slabs * nrb;
    int64_t grid = blocks;
    if (grid > items) grid = items;
    if (grid > kMaxFitBlocks) grid = kMaxFitBlocks;
    int64_t per_block = (items + grid - 1) / grid;
    p.tail_item0 = (int)items;
    p.tail_quarters = 0;
    {
        // an even number of whole items per block plus a quarter-item tail, where that is shorter for
        // the busiest block (a tail row costs more than a quarter of a pipelined item: count it double)
        const int64_t g = blocks < kMaxFitBlocks ? blocks : kMaxFitBlocks;
        const int64_t whole = items / g, rest = items - whole * g;
        if (whole >= 4 && rest > 0 && 4 * rest <= g && 2 * whole + 1 < 2 * per_block) {
            per_block = whole;
            p.tail_item0 = (int)(whole * g);
            p.tail_quarters = (int)(4 * rest);
            grid = g;
        }
    }
    if (p.tail_quarters == 0) grid = (items + per_block - 1) / per_block;
    p.nrb = (int)nrb; p.items = (int)items; p.per_block = (int)per_block;
    p.arrivals = (unsigned)grid + (unsigned)g_extra_arrivals;
    return grid;
}

static bool fill_params(FitParams& p, const FitLayerArgs& a, int n_outer, uint32_t* dev_status) {
    p = FitParams{};
    p.W = a.W; p.N = a.N; p.K = a.K; p.ldw = a.ldw;
    p.scales = static_cast<const uint8_t*>(a.scales); p.rinv = a.ws.rinv; p.I = a.I;
    p.ctrl = a.ws.ctrl; p.acc = reinterpret_cast<unsigned long long*>(a.ws.part); p.err_trace = a.err_trace; p.T01_out = a.T01_out; p.dev_status = dev_status;
    p.n_rounds = n_outer; p.trace_base = 0; p.bar_base = 0u;
    p.spin_limit = g_spin_limit;
    p.sigw = a.ws.qlist;            // the quantile selection's list is free once the start tables exist
    const int64_t slabs = (a.K + 255) / 256;
    constexpr int kRowsPerItem = kRowsPerWarp * AAAC_FIT_WARPS;
    const int64_t nrb = (a.N + kRowsPerItem - 1) / kRowsPerItem;
    return !(a.N > 0x7FFFFFFF || a.K > 0x7FFFFFFF || slabs * nrb > 0x7FFFFFFF);
}

cudaError_t launch_fit_rounds(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int sel_group, const void* scales,
                              const float* I, int n_outer, int n_inner, double* err_trace, float* T01_out, uint32_t* dev_status,
                              const Workspace& ws, cudaStream_t st) {
    if (n_outer <= 0) return cudaSuccess;
    if (n_inner < 1 || (int64_t)n_outer * n_inner > 0x7FFFFFFF) return cudaErrorInvalidValue;
    FitLayerArgs a{W, N, K, ldw, scales, I, err_trace, T01_out, ws};
    FitParams p;
    if (!fill_params(p, a, n_outer, dev_status)) return cudaErrorInvalidValue;
    const int64_t grid = plan_layer(p, N, K, sm_count());
    constexpr int NW = AAAC_FIT_WARPS, REP = AAAC_FIT_REP;
    auto launch = [&](auto kind) {
        constexpr int KIND = decltype(kind)::value;
        if (mode == AAAC_INT4 && sel_group == 16) return launch_variant<AAAC_INT4, 16, NW, REP, KIND>(p, (unsigned)grid, st);
        if (mode == AAAC_INT4) return launch_variant<AAAC_INT4, 128, NW, REP, KIND>(p, (unsigned)grid, st);
        return launch_variant<AAAC_NVFP4, 16, NW, REP, KIND>(p, (unsigned)grid, st);
    };
    // the three rotating sum buffers start at zero
    static_assert(sizeof(unsigned long long) * 3 * kAccBuffer <= sizeof(double) * kMaxBlocks * kPartStride, "the sum buffers live in the block-partial region");
    cudaError_t em = cudaMemsetAsync(p.acc, 0, sizeof(unsigned long long) * 3 * kAccBuffer, st);
    if (em != cudaSuccess) return em;
    if (n_inner == 1) return launch(std::integral_constant<int, kRounds>{});
    for (int outer = 0; outer < n_outer; ++outer) {
        p.n_rounds = 1; p.trace_base = outer;
        cudaError_t e = launch(std::integral_constant<int, kAssignKeep>{});
        if (e != cudaSuccess) return e;
        p.bar_base += 1u;
        p.n_rounds = n_inner - 1;
        e = launch(std::integral_constant<int, kInner>{});
        if (e != cudaSuccess) return e;
        p.bar_base += (unsigned)(n_inner - 1);
    }
    return cudaSuccess;
}

template <int MODE, int SEL>
static cudaError_t launch_batch_variant(FitBatch& b, unsigned grid, cudaStream_t st) {
    constexpr int NW = AAAC_FIT_WARPS, REP = AAAC_FIT_REP;
    auto kern = fit_batch_kernel<MODE, SEL, NW, REP>;
    size_t smem = 0;
    cudaError_t e = fit_dynamic_smem(reinterpret_cast<const void*>(kern), &smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    void* args[] = {&b};
    note_launch();
    // cooperative: the blocks of a layer wait for each other, so all of them must be resident
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kern), dim3(grid), dim3(NW * 32), args, smem, st);
}

cudaError_t launch_fit_rounds_batch(const FitLayerArgs* layers, int n, int mode, int sel_group, int n_outer, int n_inner,
                                    uint32_t* dev_status, cudaStream_t st) {
    if (n_outer <= 0 || n <= 0) return cudaSuccess;
    if (n_inner < 1 || (int64_t)n_outer * n_inner > 0x7FFFFFFF) return cudaErrorInvalidValue;
    const int sms = sm_count();
    for (int at = 0; at < n;) {
        const int m = (n - at) < kMaxBatch ? (n - at) : kMaxBatch;
        if (m == 1 || n_inner > 1 || m > sms) {
            // single layers and inner refinement go through the one-layer launches
            const FitLayerArgs& a = layers[at];
            cudaError_t e = launch_fit_rounds(a.W, a.N, a.K, a.ldw, mode, sel_group, a.scales, a.I, n_outer, n_inner,
                                              a.err_trace, a.T01_out, dev_status, a.ws, st);
            if (e != cudaSuccess) return e;
            at += 1;
            continue;
        }
        FitBatch b{};
        int64_t items[kMaxBatch], share[kMaxBatch];
        constexpr int kRowsPerItem = kRowsPerWarp * AAAC_FIT_WARPS;
        for (int l = 0; l < m; ++l) {
            const FitLayerArgs& a = layers[at + l];
            if (!fill_params(b.L[l], a, n_outer, dev_status)) return cudaErrorInvalidValue;
            items[l] = ((a.K + 255) / 256) * ((a.N + kRowsPerItem - 1) / kRowsPerItem);
            share[l] = 1;
        }
        // one block per layer, then every further block to the layer whose busiest block has the most items
        for (int left = sms - m; left > 0; --left) {
            int best = -1;
            int64_t load = 0;
            for (int l = 0; l < m; ++l) {
                const int64_t per = (items[l] + share[l] - 1) / share[l];
                if (share[l] < items[l] && share[l] < kMaxFitBlocks && per > load) { load = per; best = l; }
            }
            if (best < 0) break;
            ++share[best];
        }
        unsigned grid = 0;
        for (int l = 0; l < m; ++l) {
            const FitLayerArgs& a = layers[at + l];
            b.first[l] = grid;
            grid += (unsigned)plan_layer(b.L[l], a.N, a.K, share[l]);
            cudaError_t em = cudaMemsetAsync(b.L[l].acc, 0, sizeof(unsigned long long) * 3 * kAccBuffer, st);
            if (em != cudaSuccess) return em;
        }
        for (int l = m; l <= kMaxBatch; ++l) b.first[l] = grid;
        cudaError_t e;
        if (mode == AAAC_INT4 && sel_group == 16) e = launch_batch_variant<AAAC_INT4, 16>(b, grid, st);
        else if (mode == AAAC_INT4) e = launch_batch_variant<AAAC_INT4, 128>(b, grid, st);
        else e = launch_batch_variant<AAAC_NVFP4, 16>(b, grid, st);
        if (e != cudaSuccess) return e;
        at += m;
    }
    return cudaSuccess;
}

void set_fit_wait(int extra_arrivals, unsigned spin_limit) {
    g_extra_arrivals = extra_arrivals > 0 ? extra_arrivals : 0;
    g_spin_limit = spin_limit ? spin_limit : kDefaultSpinLimit;
}

cudaError_t launch_export_tables(float* T01, const Workspace& ws, cudaStream_t st) {
    export_tables_kernel<<<1, 32, 0, st>>>(ws.ctrl, T01);
    note_launch();
    return cudaGetLastError();
}

}  // namespace aaac
