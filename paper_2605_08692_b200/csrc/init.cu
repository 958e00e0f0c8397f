// Initial tables (Algorithm 1 lines 4-5).
//
// Quantile initialisation (Eq. 9, Eq. 10): T0[i] = Quantile_{i/15}, T1[i] = Quantile_{d + (1-d) i/15},
// d = 1/30, of all N*K normalised weights, with linear interpolation at position q (n - 1).
// That needs up to 64 exact order statistics of n values.  They are selected without sorting:
//   1. histogram of every w~ over 16384 uniform bins on [-8, 8) (shared-memory histogram per
//      block, merged with integer atomics);
//   2. one block turns the histogram into a prefix sum, finds the bin and the rank inside the
//      bin of every requested order statistic, and gives each distinct bin a slot;
//   3. a second pass over W appends the (order-preserving integer keys of the) values that fall
//      into a slotted bin to that slot's list -- the lists' sizes are known from step 1.  A block
//      stages its candidates in shared memory and reserves list space once per slot, so the
//      global counters see one atomic per block and slot instead of one per candidate;
//   4. one block per slot selects the requested ranks of its list by an 8-bit radix select (the
//      list is read once into registers when it is short enough, else streamed per pass);
//   5. the table entries are interpolated in double and rounded to FP32.
// Integer atomics only, so the result does not depend on scheduling.
//
// Grid initialisation: T0 = the format's table (INT4: -8..7, NVFP4: signed E2M1 with both
// zeros), T1[i] = (T0[i] + T0[i+1]) / 2 and T1[15] = T0[15] + (T0[15] - T0[14]) / 2.
#include "internal.cuh"

namespace aaac {

namespace {

__device__ __forceinline__ uint32_t float_key(float f) {      // order-preserving; -0 and +0 share a key
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
constexpr uint32_t kSlotOver = 0x40u;      // bin -> slot table: the slot's candidates have no room in the list
__device__ __forceinline__ float key_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}
// reciprocal of the group's scale for the 8 weights a lane holds
template <int MODE>
__device__ __forceinline__ float group_rinv(const void* scales, int64_t gi, float s_t) {
    if (MODE == AAAC_INT4) {
        const uint32_t b = reinterpret_cast<const uint16_t*>(scales)[gi] & 0x7FFFu;
        return __frcp_rn(__uint_as_float(b << 16));
    }
    const uint32_t c = reinterpret_cast<const uint8_t*>(scales)[gi] & 0x7Fu;
    return __frcp_rn(__fmul_rn(e4m3_value(c), s_t));
}

// Step 1: histogram of every w~ (shared-memory counters per block, merged with integer atomics).
// A warp takes four 256-column pieces per iteration so that four loads are in flight.
template <int MODE>
__global__ void __launch_bounds__(512, 3)
quantile_hist_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw,
                     const void* __restrict__ scales, const Ctrl* ctrl, uint32_t* __restrict__ hist) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    extern __shared__ uint32_t sm[];                      // kQBins counters
    const int lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kQBins; i += blockDim.x) sm[i] = 0;
    __syncthreads();
    const float s_t = ctrl->s_t;
    const int64_t slabs = (K + 255) / 256, Gr = K / G;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    SlabWalk it(warp0, nwarps, slabs);
    while (it.row < N) {
        uint4 v[4];
        float r[4];
        bool ok[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int64_t row = it.row, col = (int64_t)it.slab * 256 + lane * 8;
            ok[h] = row < N && col < K;
            v[h] = make_uint4(0, 0, 0, 0);
            r[h] = 0.f;
            if (ok[h]) {
                v[h] = __ldg(reinterpret_cast<const uint4*>(W + row * ldw + col));
                r[h] = group_rinv<MODE>(scales, row * Gr + col / G, s_t);
            }
            it.next();
        }
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            if (!ok[h]) continue;
            const uint32_t w[4] = {v[h].x, v[h].y, v[h].z, v[h].w};
#pragma unroll
            for (int j = 0; j < 8; ++j)
                atomicAdd(&sm[qbin(__fmul_rn((j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]), r[h]))], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kQBins; i += blockDim.x)
        if (sm[i]) atomicAdd(&hist[i], sm[i]);
}

// Step 3: candidates of the slotted bins, staged per block.
constexpr int kStageCap = 4096;                  // staged candidates per block
constexpr int kStageEvery = 4;                   // loop iterations between two looks at the stage's fill

template <int MODE>
__global__ void __launch_bounds__(256)
quantile_collect_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw,
                        const void* __restrict__ scales, Ctrl* ctrl, const uint8_t* __restrict__ slot_of_bin,
                        uint32_t* __restrict__ list) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    extern __shared__ uint32_t sm[];                      // kQBins bytes of slot ids
    __shared__ uint32_t buf_key[kStageCap];
    __shared__ uint8_t buf_slot[kStageCap];
    __shared__ uint16_t buf_pos[kStageCap];
    __shared__ uint32_t cnt[kQReq];
    __shared__ unsigned long long base[kQReq];
    __shared__ uint32_t nbuf;
    __shared__ uint32_t okmin[kQReq], okmax[kQReq];       // smallest / largest key of the slots without list space
    __shared__ float rl[128];                             // NVFP4: reciprocal of the effective scale per E4M3 code
    const int tid = threadIdx.x, lane = tid & 31;
    const float s_t = ctrl->s_t;
    if (MODE == AAAC_NVFP4 && tid < 128) rl[tid] = __frcp_rn(__fmul_rn(e4m3_value((uint32_t)tid), s_t));
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(slot_of_bin);
        for (int i = tid; i < kQBins / 4; i += blockDim.x) sm[i] = src[i];
        if (tid == 0) nbuf = 0;
        if (tid < kQReq) { okmin[tid] = 0xFFFFFFFFu; okmax[tid] = 0u; }
    }
    __syncthreads();
    const uint8_t* sm_slot = reinterpret_cast<const uint8_t*>(sm);
    const int64_t slabs = (K + 255) / 256, items = N * slabs, Gr = K / G;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + tid) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t iters = (items + 2 * nwarps - 1) / (2 * nwarps);     // two items per warp and iteration

    auto flush = [&]() {                                  // called by the whole block, after a barrier
        const uint32_t n = min(nbuf, (uint32_t)kStageCap);
        if (tid < kQReq) cnt[tid] = 0;
        __syncthreads();
        for (uint32_t i = tid; i < n; i += blockDim.x) buf_pos[i] = (uint16_t)atomicAdd(&cnt[buf_slot[i]], 1u);
        __syncthreads();
        if (tid < kQReq && cnt[tid])
            base[tid] = ctrl->slot_off[tid] + atomicAdd(&ctrl->slot_fill[tid], cnt[tid]);
        __syncthreads();
        for (uint32_t i = tid; i < n; i += blockDim.x) list[base[buf_slot[i]] + buf_pos[i]] = buf_key[i];
        __syncthreads();
        if (tid == 0) nbuf = 0;
        __syncthreads();
    };

    SlabWalk it(warp0, nwarps, slabs);
    // (the scale travels as its stored bits: nothing waits for the load before the row is worked on)
    auto fetch = [&](uint4& vv, uint32_t& ss, bool& okk) {
        const int64_t row = it.row, col = (int64_t)it.slab * 256 + lane * 8;
        okk = row < N && col < K;
        vv = make_uint4(0, 0, 0, 0);
        ss = 0u;
        if (okk) {
            vv = __ldg(reinterpret_cast<const uint4*>(W + row * ldw + col));
            const int64_t gi = row * Gr + col / G;
            if (MODE == AAAC_INT4) ss = reinterpret_cast<const uint16_t*>(scales)[gi];
            else ss = reinterpret_cast<const uint8_t*>(scales)[gi];
        }
        it.next();
    };
    // The slots of a lane's eight weights first.  A slot byte has bit 7 set where the bin is not asked
    // for, so the AND of the eight bytes tells whether the lane holds a candidate; a lane that does
    // walks only its candidates (one, nearly always), found by a bit scan of the packed bytes, and
    // recomputes w~ of that weight alone.
    auto take = [&](const uint4& v, uint32_t ss) {
        // the reciprocal group_rinv would give for these scale bits
        const float r = MODE == AAAC_INT4 ? __frcp_rn(__uint_as_float((ss & 0x7FFFu) << 16)) : rl[ss & 0x7Fu];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t sl[8], all = 0x80u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            sl[j] = sm_slot[qbin(__fmul_rn((j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]), r))];
            all &= sl[j];
        }
        if (all) return;
        const uint32_t lo = __byte_perm(__byte_perm(sl[0], sl[1], 0x0040), __byte_perm(sl[2], sl[3], 0x0040), 0x5410);
        const uint32_t hi = __byte_perm(__byte_perm(sl[4], sl[5], 0x0040), __byte_perm(sl[6], sl[7], 0x0040), 0x5410);
        const uint64_t bytes = ((uint64_t)hi << 32) | lo;
        uint64_t todo = ~bytes & 0x8080808080808080ull;
        while (todo) {
            const int j = (__ffsll((long long)todo) - 1) >> 3;
            todo &= todo - 1;
            const uint32_t s = (uint32_t)(bytes >> (8 * j)) & 0xFFu;
            const uint32_t ww = (j >> 1) == 0 ? w[0] : (j >> 1) == 1 ? w[1] : (j >> 1) == 2 ? w[2] : w[3];
            const uint32_t key = float_key(__fmul_rn((j & 1) ? bf16_hi(ww) : bf16_lo(ww), r));
            if (s & kSlotOver) {
                // no list space for this slot: keep only the extremes of its keys (lanes with the
                // same slot combine first, so that a heavy bin costs one atomic per warp step)
                const uint32_t so = s & (kSlotOver - 1u);
                const unsigned peers = __match_any_sync(__activemask(), so);
                const uint32_t mn = __reduce_min_sync(peers, key), mx = __reduce_max_sync(peers, key);
                if (lane == __ffs(peers) - 1) { atomicMin(&okmin[so], mn); atomicMax(&okmax[so], mx); }
            } else {
                const uint32_t pos = atomicAdd(&nbuf, 1u);
                if (pos < (uint32_t)kStageCap) {
                    buf_key[pos] = key;
                    buf_slot[pos] = (uint8_t)s;
                } else {
                    // the stage is full until the block next looks at it: straight to the slot's list
                    list[ctrl->slot_off[s] + atomicAdd(&ctrl->slot_fill[s], 1u)] = key;
                }
            }
        }
    };

    // Two items per warp are in flight: the loads of iteration k + 1 are issued before iteration k
    // is processed.  The warps of a block meet only every kStageEvery iterations, to empty the
    // stage once it is half full (the vote makes the decision the same for every thread).
    uint4 va, vb;
    uint32_t ra, rb;
    bool oka, okb;
    fetch(va, ra, oka);
    fetch(vb, rb, okb);
    for (int64_t k = 0; k < iters; ++k) {
        uint4 vna, vnb;
        uint32_t rna, rnb;
        bool okna, oknb;
        fetch(vna, rna, okna);
        fetch(vnb, rnb, oknb);
        if (oka) take(va, ra);
        if (okb) take(vb, rb);
        if ((k % kStageEvery) == kStageEvery - 1 && __syncthreads_or(nbuf > (uint32_t)kStageCap / 2)) flush();
        va = vna; ra = rna; oka = okna;
        vb = vnb; rb = rnb; okb = oknb;
    }
    __syncthreads();
    flush();
    if (tid < kQReq && okmin[tid] <= okmax[tid]) {
        atomicMin(&ctrl->slot_kmin[tid], okmin[tid]);
        atomicMax(&ctrl->slot_kmax[tid], okmax[tid]);
    }
}

struct Requests {                     // the order statistics asked for (host-computed from N K alone)
    unsigned long long rank[kQReq];
    double frac[2 * kM];
};

// one block of 1024 threads: prefix sum, bin + local rank of every request, slots.  Every thread
// keeps its chunk of 16 bins in registers; the thread whose chunk holds a requested rank walks
// those registers (no dependent memory reads), and the bin -> slot table is cleared by word stores.
__global__ void __launch_bounds__(1024)
quantile_plan_kernel(Ctrl* ctrl, const uint32_t* __restrict__ hist, uint8_t* __restrict__ slot_of_bin,
                     unsigned long long qcap, const Requests rq) {
    __shared__ unsigned long long chunk[1024];
    __shared__ unsigned long long req_rank[kQReq];
    __shared__ int req_bin[kQReq];
    __shared__ unsigned long long req_cnt[kQReq];
    __shared__ int req_first[kQReq];
    __shared__ unsigned long long wtot[32];
    const int tid = threadIdx.x;
    constexpr int per = kQBins / 1024;
    static_assert(per == 16, "a thread's chunk is four 16-byte loads");
    uint32_t h[per];
    {
        const uint4* src = reinterpret_cast<const uint4*>(hist + tid * per);
#pragma unroll
        for (int i = 0; i < per / 4; ++i) {
            const uint4 v = __ldg(src + i);
            h[4 * i] = v.x; h[4 * i + 1] = v.y; h[4 * i + 2] = v.z; h[4 * i + 3] = v.w;
        }
    }
    unsigned long long s = 0;
#pragma unroll
    for (int i = 0; i < per; ++i) s += h[i];
    if (tid < kQReq) req_rank[tid] = rq.rank[tid];
    if (tid < 2 * kM) ctrl->frac[tid] = rq.frac[tid];
    if (tid == 0) ctrl->done = 0u;                          // blocks of the selection kernel that have finished
    {
        uint32_t* clr = reinterpret_cast<uint32_t*>(slot_of_bin);
#pragma unroll
        for (int i = 0; i < kQBins / 4 / 1024; ++i) clr[tid + i * 1024] = 0xFFFFFFFFu;
    }
    // exclusive prefix of the 1024 chunk sums: warp scans, then a scan of the 32 warp totals
    {
        const int lane = tid & 31, warp = tid >> 5;
        unsigned long long v = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, v, o);
            if (lane >= o) v += t;
        }
        if (lane == 31) wtot[warp] = v;
        __syncthreads();
        if (warp == 0) {
            unsigned long long w = wtot[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, w, o);
                if (lane >= o) w += t;
            }
            wtot[lane] = w;                               // inclusive
        }
        __syncthreads();
        chunk[tid] = v - s + (warp ? wtot[warp - 1] : 0ull);
    }
    __syncthreads();
    {
        // The requests whose rank lies in this thread's chunk (the last chunk also takes ranks beyond the
        // data, which are never requested).  A warp first sieves the 64 requests against the range of
        // its 32 chunks, two requests per lane, and only the few that pass are looked at by every lane;
        // the owning thread then walks its chunk's bins in registers.
        const unsigned long long lo = chunk[tid], hi = lo + s;
        const int lane = tid & 31, warp = tid >> 5;
        const unsigned long long wlo = __shfl_sync(0xFFFFFFFFu, lo, 0), whi = __shfl_sync(0xFFFFFFFFu, hi, 31);
#pragma unroll
        for (int half = 0; half < kQReq / 32; ++half) {
            const unsigned long long rq_ = req_rank[half * 32 + lane];
            unsigned mask = __ballot_sync(0xFFFFFFFFu, rq_ >= wlo && (rq_ < whi || warp == 31));
            while (mask) {
                const int q = half * 32 + __ffs(mask) - 1;
                mask &= mask - 1;
                const unsigned long long r = req_rank[q];
                if (!(r >= lo && (r < hi || tid == 1023))) continue;
                unsigned long long base = lo;
                int i = 0;
#pragma unroll
                for (int k = 0; k < per - 1; ++k)
                    if (i == k && r >= base + h[k]) { base += h[k]; ++i; }
                uint32_t hv = h[0];
#pragma unroll
                for (int k = 1; k < per; ++k) if (i == k) hv = h[k];
                req_bin[q] = tid * per + i;
                req_cnt[q] = hv;
                ctrl->req_local[q] = r - base;
            }
        }
    }
    __syncthreads();
    if (tid < kQReq) {
        // a slot per distinct bin, in order of first appearance among the requests
        int first = tid;
        for (int q = 0; q < tid; ++q)
            if (req_bin[q] == req_bin[tid]) { first = q; break; }
        req_first[tid] = first;
    }
    __syncthreads();
    // slots in order of first appearance among the requests.  A slot gets list space while the list has
    // room for all of its bin's weights; otherwise it is marked and only the extremes of its keys will
    // be kept.  When everything fits (the usual case) the 64 requests work out their slots side by side.
    __shared__ uint32_t slot_of_req[kQReq];
    __shared__ int all_fit;
    if (tid < kQReq) {
        uint32_t slot = 0, ns = 0;
        unsigned long long off = 0, tot = 0;
        const int first = req_first[tid];
        for (int q = 0; q < kQReq; ++q) {
            if (req_first[q] != q) continue;
            if (q < first) { ++slot; off += req_cnt[q]; }
            ++ns;
            tot += req_cnt[q];
        }
        if (tid == 0) all_fit = tot <= qcap;
        if (tot <= qcap) {
            slot_of_req[tid] = slot;
            if (first == tid) {
                ctrl->slot_off[slot] = off;
                ctrl->slot_fill[slot] = 0;
                ctrl->slot_over[slot] = 0u;
                slot_of_bin[req_bin[tid]] = (uint8_t)slot;
            }
            if (tid == kQReq - 1) {
                ctrl->slot_off[ns] = tot;
                ctrl->nslots = ns;
                ctrl->scratch_short = 0u;
            }
        }
    }
    __syncthreads();
    if (tid == 0 && !all_fit) {
        uint32_t ns = 0;
        unsigned long long off = 0;
        for (int q = 0; q < kQReq; ++q) {
            if (req_first[q] != q) { slot_of_req[q] = slot_of_req[req_first[q]]; continue; }
            const bool fits = off + req_cnt[q] <= qcap;
            slot_of_req[q] = ns;
            ctrl->slot_off[ns] = off;
            ctrl->slot_fill[ns] = 0;
            ctrl->slot_over[ns] = fits ? 0u : 1u;
            ctrl->slot_kmin[ns] = 0xFFFFFFFFu;
            ctrl->slot_kmax[ns] = 0u;
            slot_of_bin[req_bin[q]] = (uint8_t)(fits ? ns : (ns | kSlotOver));
            if (fits) off += req_cnt[q];
            ++ns;
        }
        ctrl->slot_off[ns] = off;
        ctrl->nslots = ns;
        ctrl->scratch_short = 0u;
    }
    __syncthreads();
    if (tid < kQReq) ctrl->req_slot[tid] = slot_of_req[tid];
}

// one block per slot: radix select of every request that lives in this slot.
//  - The first kKeep * 1024 keys of the list are read once and stay in registers for every sweep;
//    only what is beyond them is streamed from memory, eight loads in flight per thread.
//  - The keys of a slot lie in one narrow bin, so they share their leading bits: one sweep finds
//    the bits on which all keys agree, and only the 8-bit digits below them need a radix pass.
//    Within a pass equal digits within a warp are counted once (match), which keeps the
//    shared-memory atomics apart.
//  - The two neighbours that one table entry interpolates between are consecutive ranks: the
//    second is the first's key again, or the smallest larger key -- one sweep instead of a
//    second selection.
__device__ __forceinline__ void select_slot(Ctrl* ctrl, const uint32_t* __restrict__ list) {
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sh_prefix, sh_mask;
    __shared__ unsigned long long sh_k;
    __shared__ uint32_t req_slot[kQReq];
    __shared__ unsigned long long req_local[kQReq];
    __shared__ uint32_t sh_or, sh_and, sh_cnt, sh_min;
    const uint32_t slot = blockIdx.x;
    if (slot >= ctrl->nslots) return;
    if (ctrl->slot_over[slot]) {
        // the bin's weights had no room in the list: if they all share one value, that value is every
        // order statistic of the bin; otherwise the scratch was too small for this layer
        const uint32_t kmin = ctrl->slot_kmin[slot], kmax = ctrl->slot_kmax[slot];
        if (threadIdx.x < kQReq && ctrl->req_slot[threadIdx.x] == slot) {
            if (kmin == kmax) ctrl->rank_val[threadIdx.x] = key_float(kmin);
            else { ctrl->rank_val[threadIdx.x] = 0.f; ctrl->scratch_short = 1u; }
        }
        return;
    }
    if (threadIdx.x < kQReq) {
        req_slot[threadIdx.x] = ctrl->req_slot[threadIdx.x];
        req_local[threadIdx.x] = ctrl->req_local[threadIdx.x];
    }
    if (threadIdx.x == 0) { sh_or = 0u; sh_and = 0xFFFFFFFFu; }
    const uint32_t* keys = list + ctrl->slot_off[slot];
    const unsigned long long n = ctrl->slot_off[slot + 1] - ctrl->slot_off[slot];
    const unsigned long long n_up = (n + blockDim.x - 1) / blockDim.x * blockDim.x;
    const int lane = threadIdx.x & 31;
    constexpr int kKeep = 24;
    const unsigned long long n_keep = min(n_up, (unsigned long long)kKeep * blockDim.x);   // a multiple of the block size
    uint32_t kc[kKeep];
#pragma unroll
    for (int u = 0; u < kKeep; ++u) {
        const unsigned long long i = threadIdx.x + (unsigned long long)u * blockDim.x;
        kc[u] = i < n ? keys[i] : 0u;
    }
    // f(key, valid) for every key of the list; every thread of the block makes the same calls
    auto for_each_key = [&](auto f) {
#pragma unroll
        for (int u = 0; u < kKeep; ++u) {
            if ((unsigned long long)u * blockDim.x >= n_keep) break;
            f(kc[u], threadIdx.x + (unsigned long long)u * blockDim.x < n);
        }
        for (unsigned long long i0 = n_keep + threadIdx.x; i0 < n_up; i0 += 8ull * blockDim.x) {
            uint32_t kk[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned long long i = i0 + (unsigned long long)u * blockDim.x;
                kk[u] = i < n ? keys[i] : 0u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned long long i = i0 + (unsigned long long)u * blockDim.x;
                if (i >= n_up) break;
                f(kk[u], i < n);
            }
        }
    };
    __syncthreads();
    {
        uint32_t o = 0u, a = 0xFFFFFFFFu;
        for_each_key([&](uint32_t k, bool valid) { if (valid) { o |= k; a &= k; } });
        o = __reduce_or_sync(0xFFFFFFFFu, o);
        a = __reduce_and_sync(0xFFFFFFFFu, a);
        if (lane == 0) { atomicOr(&sh_or, o); atomicAnd(&sh_and, a); }
    }
    __syncthreads();
    int first_shift = 24;
    uint32_t first_prefix = 0u, first_mask = 0u;
    if (n > 0) {
        const uint32_t diff = sh_or ^ sh_and;
        first_shift = diff ? ((31 - __clz(diff)) >> 3) << 3 : 0;
        first_mask = first_shift == 24 ? 0u : ~((1u << (first_shift + 8)) - 1u);
        first_prefix = sh_and & first_mask;
    }
    bool have_prev = false;                                // rank and key of the request answered last
    unsigned long long prev_k = 0;
    uint32_t prev_key = 0u;
    for (int q = 0; q < kQReq; ++q) {
        if (req_slot[q] != slot) continue;                 // uniform across the block
        if (have_prev && (req_local[q] == prev_k || req_local[q] == prev_k + 1)) {
            // the same or the next order statistic: it equals the previous key unless every key
            // up to that one is already counted, in which case it is the smallest larger key
            uint32_t key = prev_key;
            if (req_local[q] == prev_k + 1) {
                if (threadIdx.x == 0) { sh_cnt = 0u; sh_min = 0xFFFFFFFFu; }
                __syncthreads();
                uint32_t c = 0u, m = 0xFFFFFFFFu;
                for_each_key([&](uint32_t k, bool valid) {
                    if (valid) {
                        if (k <= prev_key) ++c;
                        else m = min(m, k);
                    }
                });
                c = __reduce_add_sync(0xFFFFFFFFu, c);
                m = __reduce_min_sync(0xFFFFFFFFu, m);
                if (lane == 0) { atomicAdd(&sh_cnt, c); atomicMin(&sh_min, m); }
                __syncthreads();
                if (req_local[q] >= (unsigned long long)sh_cnt && sh_min != 0xFFFFFFFFu) key = sh_min;
                __syncthreads();
            }
            if (threadIdx.x == 0) ctrl->rank_val[q] = key_float(key);
            prev_k = req_local[q];
            prev_key = key;
            continue;
        }
        if (threadIdx.x == 0) { sh_prefix = first_prefix; sh_mask = first_mask; sh_k = req_local[q]; }
        __syncthreads();
        for (int shift = first_shift; shift >= 0; shift -= 8) {
            if (threadIdx.x < 256) hist[threadIdx.x] = 0;
            __syncthreads();
            const uint32_t prefix = sh_prefix, mask = sh_mask;
            for_each_key([&](uint32_t k, bool valid) {
                const bool sel = valid && (k & mask) == prefix;
                const unsigned act = __ballot_sync(0xFFFFFFFFu, sel);
                if (sel) {
                    const uint32_t d = (k >> shift) & 0xFFu;
                    const unsigned peers = __match_any_sync(act, d);
                    if (lane == __ffs(peers) - 1) atomicAdd(&hist[d], (uint32_t)__popc(peers));
                }
            });
            __syncthreads();
            if (threadIdx.x < 32) {
                // digit that holds rank k: lane l owns digits 8 l .. 8 l + 7
                uint32_t c[8], tot = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { c[i] = hist[lane * 8 + i]; tot += c[i]; }
                uint32_t incl = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += t;
                }
                const unsigned long long k = sh_k;
                const unsigned long long before = incl - tot;
                const bool mine = k >= before && k < (unsigned long long)incl;
                const unsigned who = __ballot_sync(0xFFFFFFFFu, mine);
                // ranks beyond the list (never requested) fall to the last digit
                const int owner = who ? __ffs(who) - 1 : 31;
                if (lane == owner) {
                    unsigned long long r = k - before;
                    int i = 0;
                    for (; i < 7; ++i) {
                        if (r < c[i]) break;
                        r -= c[i];
                    }
                    sh_k = r;
                    sh_prefix = prefix | ((uint32_t)(lane * 8 + i) << shift);
                    sh_mask = mask | (0xFFu << shift);
                }
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) ctrl->rank_val[q] = key_float(sh_prefix);
        have_prev = true;
        prev_k = req_local[q];
        prev_key = sh_prefix;
        __syncthreads();
    }
}

// One block per slot; the last block to finish interpolates the table entries: entry e uses requests
// 2e (lower neighbour) and 2e+1 (upper neighbour), in double, rounded to FP32.
__global__ void __launch_bounds__(1024)
quantile_select_kernel(Ctrl* ctrl, const uint32_t* __restrict__ list, uint32_t* dev_status) {
    __shared__ int last;
    select_slot(ctrl, list);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&ctrl->done, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    const int e = threadIdx.x;
    if (e == 0) {
        ctrl->done = 0u;
        if (__ldcg(&ctrl->scratch_short) && dev_status) atomicOr(dev_status, AAAC_DEV_SCRATCH);
    }
    if (e >= 2 * kM) return;
    const double lo = (double)__ldcg(&ctrl->rank_val[2 * e]), hi = (double)__ldcg(&ctrl->rank_val[2 * e + 1]);
    const double v = __dadd_rn(lo, __dmul_rn(ctrl->frac[e], __dsub_rn(hi, lo)));
    ctrl->T[e] = (double)(float)v;
}

__global__ void grid_init_kernel(Ctrl* ctrl, int mode, const float* T01_user) {
    const int t = threadIdx.x;
    if (t >= 2 * kM) return;
    if (T01_user) {
        ctrl->T[t] = (double)T01_user[t];
        return;
    }
    const double e2m1[kM] = {-6, -4, -3, -2, -1.5, -1, -0.5, 0, 0, 0.5, 1, 1.5, 2, 3, 4, 6};
    auto base = [&](int i) { return mode == AAAC_INT4 ? (double)(i - 8) : e2m1[i]; };
    const int i = t & 15;
    if (t < kM) ctrl->T[t] = base(i);
    else ctrl->T[t] = (i < 15) ? 0.5 * (base(i) + base(i + 1)) : base(15) + 0.5 * (base(15) - base(14));
}

}  // namespace

cudaError_t launch_init(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int init,
                        const void* scales, const float* T01_user, uint32_t* dev_status, const Workspace& ws, cudaStream_t st,
                        bool hist_done) {
    if (init != AAAC_INIT_QUANTILE) {
        grid_init_kernel<<<1, 32, 0, st>>>(ws.ctrl, mode, init == AAAC_INIT_USER ? T01_user : nullptr);
        note_launch();
        return cudaGetLastError();
    }
    // positions of the 32 quantiles, as the definition states them
    Requests rq;
    const double n1 = (double)(N * K - 1);
    const double d = 1.0 / (2.0 * (kM - 1));
    for (int e = 0; e < 2 * kM; ++e) {
        const int i = e & 15;
        const double q = (e < kM) ? (double)i / (double)(kM - 1) : d + (1.0 - d) * (double)i / (double)(kM - 1);
        const double pos = q * n1;
        double lo = floor(pos), hi = ceil(pos);
        if (lo < 0) lo = 0;
        if (hi > n1) hi = n1;
        if (lo > hi) lo = hi;
        rq.rank[2 * e] = (unsigned long long)lo;
        rq.rank[2 * e + 1] = (unsigned long long)hi;
        rq.frac[e] = pos - lo;
    }
    cudaError_t e;
    const int blocks = sm_count() * 3;
    const size_t sm0 = kQBins * sizeof(uint32_t);
    if (hist_done) {
        // the scales pass has already counted the histogram (launch_scales with with_hist)
    } else if ((e = cudaMemsetAsync(ws.qhist, 0, kQBins * sizeof(uint32_t), st)) != cudaSuccess) {
        return e;
    } else if (mode == AAAC_INT4) {
        if ((e = cudaFuncSetAttribute(quantile_hist_kernel<AAAC_INT4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm0)) != cudaSuccess) return e;
        quantile_hist_kernel<AAAC_INT4><<<blocks, 512, sm0, st>>>(W, N, K, ldw, scales, ws.ctrl, ws.qhist);
        note_launch();
    } else {
        if ((e = cudaFuncSetAttribute(quantile_hist_kernel<AAAC_NVFP4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm0)) != cudaSuccess) return e;
        quantile_hist_kernel<AAAC_NVFP4><<<blocks, 512, sm0, st>>>(W, N, K, ldw, scales, ws.ctrl, ws.qhist);
        note_launch();
    }
    quantile_plan_kernel<<<1, 1024, 0, st>>>(ws.ctrl, ws.qhist, ws.qslot_of_bin, (unsigned long long)ws.qcap, rq);
    note_launch();
    const int blocks1 = sm_count() * 4;
    if (mode == AAAC_INT4)
        quantile_collect_kernel<AAAC_INT4><<<blocks1, 256, kQBins, st>>>(W, N, K, ldw, scales, ws.ctrl, ws.qslot_of_bin, ws.qlist);
    else
        quantile_collect_kernel<AAAC_NVFP4><<<blocks1, 256, kQBins, st>>>(W, N, K, ldw, scales, ws.ctrl, ws.qslot_of_bin, ws.qlist);
    note_launch();
    quantile_select_kernel<<<kQReq, 1024, 0, st>>>(ws.ctrl, ws.qlist, dev_status);
    note_launch();
    return cudaGetLastError();
}

}  // namespace aaac
