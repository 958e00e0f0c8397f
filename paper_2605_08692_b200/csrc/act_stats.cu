// Activation importance (Eq. 7): I[k] = sum_t X[t,k]^2, a streaming column reduction.
//
// Layout: X is [T x K] BF16 row-major.  A block covers 256 adjacent columns (each lane owns
// 8 of them = one 128-bit load per row) and a strip of rows; its 8 warps take rows
// round-robin.  The square of a BF16 value is exact in FP32 (16 significant bits); a thread adds
// its squares error-free into an FP32 pair (two-sum), because double-precision arithmetic runs
// at a small fraction of the FP32 rate on this GPU.  The pairs become doubles once per thread,
// so the result differs from an index-order double sum only by rounding at the 2^-48 level; a
// second kernel adds the strip partials in strip order and rounds once to FP32.
#include <mutex>

#include "internal.cuh"

namespace aaac {

namespace {

constexpr int kWarps = 8;
constexpr int kUnroll = 4;

// hi + lo += v without rounding error (Knuth's two-sum; intrinsics so that nothing is re-associated)
__device__ __forceinline__ void two_sum(float& hi, float& lo, float v) {
    const float s = __fadd_rn(hi, v);
    const float bb = __fsub_rn(s, hi);
    const float err = __fadd_rn(__fsub_rn(hi, __fsub_rn(s, bb)), __fsub_rn(v, bb));
    hi = s;
    lo = __fadd_rn(lo, err);
}
__device__ __forceinline__ void add_squares(float (&hi)[8], float (&lo)[8], uint4 v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float a = bf16_lo(w[j]), b = bf16_hi(w[j]);
        two_sum(hi[2 * j], lo[2 * j], __fmul_rn(a, a));
        two_sum(hi[2 * j + 1], lo[2 * j + 1], __fmul_rn(b, b));
    }
}

__global__ void __launch_bounds__(kWarps * 32)
act_sumsq_kernel(const uint16_t* __restrict__ X, int64_t T, int64_t K, int64_t ldx,
                 double* __restrict__ part, int rows_per_split) {
    __shared__ double sm[kWarps][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t col0 = (int64_t)blockIdx.x * 256 + lane * 8;
    const bool active = col0 < K;
    const int64_t t_begin = (int64_t)blockIdx.y * rows_per_split;
    const int64_t t_end = min(T, t_begin + rows_per_split);
    float hi[8], lo[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { hi[j] = 0.f; lo[j] = 0.f; }

    if (active) {
        const uint16_t* base = X + col0;
        int64_t t = t_begin + warp;
        for (; t + (kUnroll - 1) * kWarps < t_end; t += kUnroll * kWarps) {
            uint4 v[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                v[u] = __ldcs(reinterpret_cast<const uint4*>(base + (t + u * kWarps) * ldx));
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) add_squares(hi, lo, v[u]);
        }
        for (; t < t_end; t += kWarps) add_squares(hi, lo, __ldcs(reinterpret_cast<const uint4*>(base + t * ldx)));
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) sm[warp][lane * 8 + j] = (double)hi[j] + (double)lo[j];
    __syncthreads();
    const int64_t col = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (col < K) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += sm[w][threadIdx.x];
        part[(int64_t)blockIdx.y * K + col] = s;
    }
}

__global__ void act_final_kernel(const double* __restrict__ part, int splits, int64_t K,
                                 float* __restrict__ I, int accumulate, uint32_t* dev_status) {
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    double s = 0.0;
    for (int p = 0; p < splits; ++p) s += part[(int64_t)p * K + k];
    float v = (float)s;
    if (accumulate) v += I[k];
    I[k] = v;
    if (dev_status && !isfinite(v)) atomicOr(dev_status, AAAC_DEV_NONFINITE);
}

}  // namespace

int act_splits_max(int64_t K) {
    const int64_t bx = (K + 255) / 256;
    int64_t want = ((int64_t)sm_count() * 8 + bx - 1) / (bx > 0 ? bx : 1);
    if (want < 1) want = 1;
    return (int)(want > kActMaxSplits ? kActMaxSplits : want);
}

cudaError_t launch_act_stats(const uint16_t* X, int64_t T, int64_t K, int64_t ldx, float* I, int accumulate,
                             uint32_t* dev_status, const Workspace& ws, cudaStream_t st) {
    const int bx = (int)((K + 255) / 256);
    int64_t want = act_splits_max(K);
    int64_t max_by_rows = (T + kWarps - 1) / kWarps;
    int64_t splits = want < 1 ? 1 : want;
    if (splits > max_by_rows) splits = max_by_rows;
    if (splits > kActMaxSplits) splits = kActMaxSplits;
    int64_t rows = (T + splits - 1) / splits;
    rows = (rows + kWarps - 1) / kWarps * kWarps;
    splits = (T + rows - 1) / rows;
    act_sumsq_kernel<<<dim3(bx, (unsigned)splits), kWarps * 32, 0, st>>>(X, T, K, ldx, ws.act_part, (int)rows);
    note_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    act_final_kernel<<<(unsigned)((K + 255) / 256), 256, 0, st>>>(ws.act_part, (int)splits, K, I, accumulate, dev_status);
    note_launch();
    return cudaGetLastError();
}

}  // namespace aaac

// ---------------------------------------------------------------------------------------------
// aaac_act_stats_noalloc: the same reduction for callers that cannot hand over scratch memory.
//
// The strip partials live in a fixed array in the library's own device image instead of a
// caller workspace, so the call needs no buffer besides X and I.  The array exists once per
// GPU that loads the library and is shared by every call on that GPU.
// ---------------------------------------------------------------------------------------------
namespace aaac {
namespace {

constexpr int kNoAllocMaxK = 32768;       // widest layer input the built-in scratch covers
constexpr int kNoAllocSplits = 32;        // row strips (8 MiB of scratch in total)

static __device__ __align__(256) double g_noalloc_part[(size_t)kNoAllocSplits * kNoAllocMaxK];

std::mutex g_noalloc_mu;
double* g_noalloc_ptr[64] = {nullptr};   // device address of the array, per device ordinal

// Host code cannot use the array's name as a pointer: the name only identifies the symbol.
// Its device address is looked up once per device, with that device current.
cudaError_t noalloc_scratch(double** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        double* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_part);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace aaac

extern "C" int aaac_act_stats_noalloc(const void* X, int64_t T, int64_t K, int64_t ldx, float* I, int accumulate,
                                      uint32_t* dev_status, void* stream) {
    using namespace aaac;
    if (!X || !I) return AAAC_ERR_NULL;
    if (T < 1 || K < 1 || K % 8 || ldx < K || ldx % 8) return AAAC_ERR_SHAPE;
    if (K > kNoAllocMaxK) return AAAC_ERR_TOO_LARGE;
    if ((reinterpret_cast<uintptr_t>(X) % 16) || (reinterpret_cast<uintptr_t>(I) % 4)) return AAAC_ERR_ALIGN;
    double* part = nullptr;
    if (noalloc_scratch(&part) != cudaSuccess) return AAAC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int bx = (int)((K + 255) / 256);
    int64_t splits = ((int64_t)sm_count() * 8 + bx - 1) / bx;
    const int64_t max_by_rows = (T + kWarps - 1) / kWarps;
    if (splits > max_by_rows) splits = max_by_rows;
    if (splits > kNoAllocSplits) splits = kNoAllocSplits;
    if (splits < 1) splits = 1;
    int64_t rows = (T + splits - 1) / splits;
    rows = (rows + kWarps - 1) / kWarps * kWarps;
    splits = (T + rows - 1) / rows;
    // every partial that the second kernel reads is written by the first: nothing has to be cleared
    act_sumsq_kernel<<<dim3(bx, (unsigned)splits), kWarps * 32, 0, st>>>(static_cast<const uint16_t*>(X), T, K, ldx,
                                                                        part, (int)rows);
    note_launch();
    if (cudaGetLastError() != cudaSuccess) return AAAC_ERR_CUDA;
    act_final_kernel<<<(unsigned)((K + 255) / 256), 256, 0, st>>>(part, (int)splits, K, I, accumulate, dev_status);
    note_launch();
    return cudaGetLastError() == cudaSuccess ? AAAC_OK : AAAC_ERR_CUDA;
}
