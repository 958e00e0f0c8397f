// Per-input-channel scaling before the fit (Section 4, "Combining AAAC with AWQ": AWQ scales the
// weights first, AAAC then learns its tables on the scaled distribution).  With a positive
// multiplier a_k per input channel, W'[n][k] = bf16(w a_k) -- one FP32 multiply, rounded to
// nearest even -- and I'_k = I_k / a_k^2 (the layer's input is divided by a_k in exchange),
// formed in double and rounded once.  A pure stream: 2 bytes in, 2 bytes out per weight; each
// thread handles 8 adjacent columns of four rows per step (four 128-bit loads in flight), so its
// eight multipliers stay in registers.
#include "internal.cuh"

namespace aaac {

namespace {

__global__ void __launch_bounds__(256)
prescale_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw, const float* __restrict__ a,
                uint16_t* __restrict__ Wout, int64_t ldo, int rows_per_block) {
    const int64_t col = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
    if (col >= K) return;
    const float4 a0 = __ldg(reinterpret_cast<const float4*>(a + col));
    const float4 a1 = __ldg(reinterpret_cast<const float4*>(a + col + 4));
    const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    const int64_t r1 = min(N, r0 + rows_per_block);
    for (int64_t row = r0; row < r1; row += 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (row + u < r1) v[u] = __ldcs(reinterpret_cast<const uint4*>(W + (row + u) * ldw + col));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (row + u >= r1) break;
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t lo = f32_to_bf16_rne(__fmul_rn(bf16_lo(w[j]), av[2 * j]));
                const uint32_t hi = f32_to_bf16_rne(__fmul_rn(bf16_hi(w[j]), av[2 * j + 1]));
                o[j] = lo | (hi << 16);
            }
            __stcs(reinterpret_cast<uint4*>(Wout + (row + u) * ldo + col), make_uint4(o[0], o[1], o[2], o[3]));
        }
    }
}

__global__ void prescale_importance_kernel(const float* __restrict__ a, int64_t K, const float* __restrict__ I,
                                           float* __restrict__ Iout, uint32_t* dev_status) {
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const float ak = a[k];
    if (!(ak > 0.f) || !(ak < __int_as_float(0x7F800000))) {           // zero, negative, infinite or NaN
        if (dev_status) atomicOr(dev_status, AAAC_DEV_NONFINITE);
    }
    if (I && Iout) Iout[k] = (float)__ddiv_rn((double)I[k], __dmul_rn((double)ak, (double)ak));
}

}  // namespace

cudaError_t launch_prescale(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, const float* a, uint16_t* Wout,
                            int64_t ldo, const float* I, float* Iout, uint32_t* dev_status, cudaStream_t st) {
    const unsigned bx = (unsigned)((K / 8 + 255) / 256);
    // enough row strips to fill the GPU a few times over, each a multiple of four rows
    int64_t strips = ((int64_t)sm_count() * 8 + bx - 1) / bx;
    if (strips > (N + 3) / 4) strips = (N + 3) / 4;
    if (strips > 65535) strips = 65535;
    if (strips < 1) strips = 1;
    int64_t rows = (N + strips - 1) / strips;
    rows = (rows + 3) / 4 * 4;
    strips = (N + rows - 1) / rows;
    prescale_kernel<<<dim3(bx, (unsigned)strips), 256, 0, st>>>(W, N, K, ldw, a, Wout, ldo, (int)rows);
    note_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    prescale_importance_kernel<<<(unsigned)((K + 255) / 256), 256, 0, st>>>(a, K, I, Iout, dev_status);
    note_launch();
    return cudaGetLastError();
}

}  // namespace aaac
