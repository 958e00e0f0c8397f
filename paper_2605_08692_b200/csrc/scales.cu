// Per-group positive scales (Algorithm 1, line 1).
//
//   INT4  (g = 128): s = bf16_rne(absmax / 7), 1 for an all-zero group, never below 2^-126.
//                    Also writes r = fl32(1/s) per group for the fit rounds.
//   NVFP4 (g = 16) : s_t = layer absmax / 2688 (a first pass over W), then per group
//                    q = E4M3_rne(absmax / (6 s_t)) kept inside 0x01..0x7E; in the lowest
//                    subnormal step the code is raised so that |w / s| <= 7.5.
// Both rules keep every normalised weight strictly inside (-8, 8).
//
// One warp handles 256 adjacent columns of one row (one 128-bit load per lane); the group
// maximum is a shuffle reduction over the 16 (INT4) or 2 (NVFP4) lanes of the group.
#include "internal.cuh"

namespace aaac {

namespace {

__device__ __forceinline__ uint32_t absmax16(uint4 v) {
    // max over the eight BF16 magnitudes (bit patterns of non-negative floats order like ints)
    uint32_t m = 0;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        m = max(m, w[j] & 0x7FFFu);
        m = max(m, (w[j] >> 16) & 0x7FFFu);
    }
    return m;
}

__global__ void __launch_bounds__(256)
absmax_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw, Ctrl* ctrl, uint32_t* dev_status) {
    const int lane = threadIdx.x & 31;
    const int64_t slabs = (K + 255) / 256;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    uint32_t m = 0;
    // four independent loads in flight per thread
    SlabWalk it(warp0, nwarps, slabs);
    while (it.row < N) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            v[u] = make_uint4(0, 0, 0, 0);
            const int64_t col = (int64_t)it.slab * 256 + lane * 8;
            if (it.row < N && col < K) v[u] = __ldg(reinterpret_cast<const uint4*>(W + (int64_t)it.row * ldw + col));
            it.next();
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) m = max(m, absmax16(v[u]));
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (lane == 0 && m) {
        atomicMax(&ctrl->absmax_bits, m << 16);
        if (m >= 0x7F80u) {
            atomicOr(&ctrl->nonfinite, 1u);
            if (dev_status) atomicOr(dev_status, AAAC_DEV_NONFINITE);
        }
    }
}

template <int MODE>
__global__ void __launch_bounds__(256)
scales_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw, void* __restrict__ scales,
              float* __restrict__ rinv, float* __restrict__ tensor_scale, Ctrl* ctrl, uint32_t* dev_status) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    constexpr int LPG = G / 8;                         // lanes per group
    const int lane = threadIdx.x & 31;
    const int64_t slabs = (K + 255) / 256, Gr = K / G;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;

    float s_t = 1.f, d6 = 6.f;
    if (MODE == AAAC_NVFP4) {
        const float A = __uint_as_float(ctrl->absmax_bits);
        s_t = (A == 0.f) ? 1.f : __fdiv_rn(A, 2688.f);
        if (s_t < 0x1p-96f) s_t = 0x1p-96f;
        d6 = __fmul_rn(6.f, s_t);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctrl->s_t = s_t;
        if (tensor_scale) tensor_scale[0] = s_t;
    }
    bool bad = false;
    SlabWalk it(warp0, nwarps, slabs);
    while (it.row < N) {
      // four independent loads in flight per thread (the row of an item is the same in every lane)
      uint4 v[4];
      int rows[4], cols[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
          v[u] = make_uint4(0, 0, 0, 0);
          rows[u] = it.row;
          cols[u] = it.slab * 256 + lane * 8;
          if (it.row < N && cols[u] < K) v[u] = __ldg(reinterpret_cast<const uint4*>(W + (int64_t)it.row * ldw + cols[u]));
          it.next();
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (rows[u] >= N) break;                       // uniform over the warp
        const int64_t row = rows[u], col = cols[u];
        uint32_t m = absmax16(v[u]);
#pragma unroll
        for (int o = LPG / 2; o; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        if (col < K && (lane % LPG) == 0) {
            const float a = __uint_as_float(m << 16);
            bad |= (m >= 0x7F80u);
            const int64_t gi = row * Gr + col / G;
            if (MODE == AAAC_INT4) {
                float s = 1.f;
                if (a != 0.f) {
                    s = __uint_as_float(f32_to_bf16_rne(__fdiv_rn(a, 7.f)) << 16);
                    if (s < 0x1p-126f) s = 0x1p-126f;
                }
                reinterpret_cast<uint16_t*>(scales)[gi] = (uint16_t)(__float_as_uint(s) >> 16);
                rinv[gi] = __frcp_rn(s);
            } else {
                const float x = __fdiv_rn(a, d6);
                uint32_t q = e4m3_encode(x);
                if (q <= 1u) q = (x > 1.25f * 0x1p-9f) ? 2u : 1u;
                reinterpret_cast<uint8_t*>(scales)[gi] = (uint8_t)q;
            }
        }
      }
    }
    if (bad) {
        atomicOr(&ctrl->nonfinite, 1u);
        if (dev_status) atomicOr(dev_status, AAAC_DEV_NONFINITE);
    }
}

// The same pass that also counts the quantile start's histogram (Eq. 9-10 need order statistics of all
// w~ = fl32(w * fl32(1/s)); their first step is a 16384-bin histogram): every lane of a group holds the
// group's maximum after the butterfly, forms the scale and its reciprocal itself -- with exactly the
// expressions the later passes use -- and bins its eight normalised weights into the block's
// shared-memory histogram, which is merged into the global one at the end.
#ifndef AAAC_SH_BLOCKS
#define AAAC_SH_BLOCKS 2
#endif
template <int MODE>
__global__ void __launch_bounds__(512, AAAC_SH_BLOCKS)
scales_hist_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw, void* __restrict__ scales,
                   float* __restrict__ rinv, float* __restrict__ tensor_scale, Ctrl* ctrl, uint32_t* dev_status,
                   uint32_t* __restrict__ hist) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    constexpr int LPG = G / 8;                         // lanes per group
    extern __shared__ uint32_t sm[];                   // kQBins counters
    for (int i = threadIdx.x; i < kQBins; i += blockDim.x) sm[i] = 0;
    const int lane = threadIdx.x & 31;
    const int64_t slabs = (K + 255) / 256, Gr = K / G;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;

    float s_t = 1.f, d6 = 6.f;
    if (MODE == AAAC_NVFP4) {
        const float A = __uint_as_float(ctrl->absmax_bits);
        s_t = (A == 0.f) ? 1.f : __fdiv_rn(A, 2688.f);
        if (s_t < 0x1p-96f) s_t = 0x1p-96f;
        d6 = __fmul_rn(6.f, s_t);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctrl->s_t = s_t;
        if (tensor_scale) tensor_scale[0] = s_t;
    }
    __shared__ float rl[128];                          // NVFP4: fl32(1 / (E4M3 value * s_t)) per scale code, as the later passes form it
    if (MODE == AAAC_NVFP4 && threadIdx.x < 128) rl[threadIdx.x] = __frcp_rn(__fmul_rn(e4m3_value(threadIdx.x), s_t));
    __syncthreads();
    bool bad = false;
    SlabWalk it(warp0, nwarps, slabs);
    while (it.row < N) {
      uint4 v[4];
      int rows[4], cols[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
          v[u] = make_uint4(0, 0, 0, 0);
          rows[u] = it.row;
          cols[u] = it.slab * 256 + lane * 8;
          if (it.row < N && cols[u] < K) v[u] = __ldg(reinterpret_cast<const uint4*>(W + (int64_t)it.row * ldw + cols[u]));
          it.next();
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (rows[u] >= N) break;                       // uniform over the warp
        const int64_t row = rows[u], col = cols[u];
        uint32_t m = absmax16(v[u]);
#pragma unroll
        for (int o = LPG / 2; o; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        if (col >= K) continue;
        const float a = __uint_as_float(m << 16);
        bad |= (m >= 0x7F80u);
        const int64_t gi = row * Gr + col / G;
        float r;                                       // fl32(1 / s), as the later passes form it
        if (MODE == AAAC_INT4) {
            float s = 1.f;
            if (a != 0.f) {
                s = __uint_as_float(f32_to_bf16_rne(__fdiv_rn(a, 7.f)) << 16);
                if (s < 0x1p-126f) s = 0x1p-126f;
            }
            r = __frcp_rn(s);
            if ((lane % LPG) == 0) {
                reinterpret_cast<uint16_t*>(scales)[gi] = (uint16_t)(__float_as_uint(s) >> 16);
                rinv[gi] = r;
            }
        } else {
            const float x = __fdiv_rn(a, d6);
            uint32_t q = e4m3_encode(x);
            if (q <= 1u) q = (x > 1.25f * 0x1p-9f) ? 2u : 1u;
            r = rl[q];
            if ((lane % LPG) == 0) reinterpret_cast<uint8_t*>(scales)[gi] = (uint8_t)q;
        }
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int j = 0; j < 8; ++j)
            atomicAdd(&sm[qbin(__fmul_rn((j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]), r))], 1u);
      }
    }
    if (bad) {
        atomicOr(&ctrl->nonfinite, 1u);
        if (dev_status) atomicOr(dev_status, AAAC_DEV_NONFINITE);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kQBins; i += blockDim.x)
        if (sm[i]) atomicAdd(&hist[i], sm[i]);
}

}  // namespace

cudaError_t launch_scales(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, void* scales,
                          float* tensor_scale, uint32_t* dev_status, const Workspace& ws, cudaStream_t st, bool with_hist) {
    const int blocks = sm_count() * 8;
    if (mode == AAAC_NVFP4) {
        absmax_kernel<<<blocks, 256, 0, st>>>(W, N, K, ldw, ws.ctrl, dev_status);
        note_launch();
    }
    if (with_hist) {
        cudaError_t e = cudaMemsetAsync(ws.qhist, 0, kQBins * sizeof(uint32_t), st);
        if (e != cudaSuccess) return e;
        const int hb = sm_count() * AAAC_SH_BLOCKS;
        const size_t sm0 = kQBins * sizeof(uint32_t);
        if (mode == AAAC_NVFP4) {
            if ((e = cudaFuncSetAttribute(scales_hist_kernel<AAAC_NVFP4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm0)) != cudaSuccess) return e;
            scales_hist_kernel<AAAC_NVFP4><<<hb, 512, sm0, st>>>(W, N, K, ldw, scales, nullptr, tensor_scale, ws.ctrl, dev_status, ws.qhist);
        } else {
            if ((e = cudaFuncSetAttribute(scales_hist_kernel<AAAC_INT4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm0)) != cudaSuccess) return e;
            scales_hist_kernel<AAAC_INT4><<<hb, 512, sm0, st>>>(W, N, K, ldw, scales, ws.rinv, tensor_scale, ws.ctrl, dev_status, ws.qhist);
        }
        note_launch();
    } else if (mode == AAAC_NVFP4) {
        scales_kernel<AAAC_NVFP4><<<blocks, 256, 0, st>>>(W, N, K, ldw, scales, nullptr, tensor_scale, ws.ctrl, dev_status);
        note_launch();
    } else {
        scales_kernel<AAAC_INT4><<<blocks, 256, 0, st>>>(W, N, K, ldw, scales, ws.rinv, tensor_scale, ws.ctrl, dev_status);
        note_launch();
    }
    return cudaGetLastError();
}

}  // namespace aaac
