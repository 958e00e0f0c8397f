// Dequantisation (Eq. 5): w^ = T_sigma[c] * s, with sigma the sign bit of the stored scale (or,
// when the selection group is 16 inside a scale group of 128, the group's bit of the separate
// selection bytes) and s the scale's magnitude (times the tensor scale for NVFP4).  A pure stream: 0.5 byte of codes and a
// scale per group in, 2 bytes out per weight.  Each thread expands one 32-bit word of codes
// (8 weights) into one 128-bit store.
#include "internal.cuh"

namespace aaac {

namespace {

template <int MODE, bool SEP>
__global__ void __launch_bounds__(256)
dequant_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales,
               const uint8_t* __restrict__ sigma_bits, const float* __restrict__ tensor_scale, const uint16_t* __restrict__ Tb,
               int64_t N, int64_t K, uint16_t* __restrict__ What, int64_t ldo) {
    constexpr int G = MODE == AAAC_INT4 ? 128 : 16;
    __shared__ float T[2 * kM];
    __shared__ float slut[128];
    if (threadIdx.x < 2 * kM) T[threadIdx.x] = __uint_as_float((uint32_t)Tb[threadIdx.x] << 16);
    if (MODE == AAAC_NVFP4 && threadIdx.x >= 128)
        slut[threadIdx.x - 128] = __fmul_rn(e4m3_value(threadIdx.x - 128), tensor_scale[0]);
    __syncthreads();
    const int64_t per_row = K / 8, Gr = K / G;
    // two independent items in flight per thread, no division per item
    SlabWalk it((int64_t)blockIdx.x * blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x, per_row);
    while (it.row < N) {
        int64_t rows[2], cols[2];
        uint32_t words[2], sb[2], sgb[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            rows[u] = it.row;
            cols[u] = (int64_t)it.slab * 8;
            words[u] = 0u; sb[u] = 0u; sgb[u] = 0u;
            if (it.row < N) {
                const int64_t row = rows[u], col = cols[u];
                words[u] = __ldcs(reinterpret_cast<const uint32_t*>(codes + ((row * K + col) >> 1)));
                const int64_t gi = row * Gr + col / G;
                sb[u] = MODE == AAAC_INT4 ? (uint32_t)reinterpret_cast<const uint16_t*>(scales)[gi]
                                          : (uint32_t)reinterpret_cast<const uint8_t*>(scales)[gi];
                if (SEP) sgb[u] = sigma_bits[row * (K >> 7) + (col >> 7)];
            }
            it.next();
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (rows[u] >= N) break;
            const int64_t row = rows[u], col = cols[u];
            const uint32_t word = words[u], b = sb[u];
            uint32_t sigma;
            float s;
            if (MODE == AAAC_INT4) {
                sigma = b >> 15;
                s = __uint_as_float((b & 0x7FFFu) << 16);
            } else {
                sigma = b >> 7;
                s = slut[b & 0x7Fu];
            }
            if (SEP) sigma = (sgb[u] >> ((col >> 4) & 7)) & 1u;
            const float* Ts = T + sigma * kM;
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // two products rounded to BF16 (nearest even) and packed by one conversion instruction
                const float lo = __fmul_rn(Ts[(word >> (8 * j)) & 15u], s);
                const float hi = __fmul_rn(Ts[(word >> (8 * j + 4)) & 15u], s);
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[j]) : "f"(hi), "f"(lo));
            }
            __stcs(reinterpret_cast<uint4*>(What + row * ldo + col), make_uint4(o[0], o[1], o[2], o[3]));
        }
    }
}

}  // namespace

cudaError_t launch_dequant(const uint8_t* codes, const void* scales, const uint8_t* sigma_bits,
                           const float* tensor_scale, const uint16_t* Tb, int64_t N, int64_t K, int mode,
                           uint16_t* What, int64_t ldo, cudaStream_t st) {
    const int64_t total = N * (K / 8);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    if (mode == AAAC_INT4 && sigma_bits)
        dequant_kernel<AAAC_INT4, true><<<(unsigned)blocks, 256, 0, st>>>(codes, scales, sigma_bits, tensor_scale, Tb, N, K, What, ldo);
    else if (mode == AAAC_INT4)
        dequant_kernel<AAAC_INT4, false><<<(unsigned)blocks, 256, 0, st>>>(codes, scales, nullptr, tensor_scale, Tb, N, K, What, ldo);
    else
        dequant_kernel<AAAC_NVFP4, false><<<(unsigned)blocks, 256, 0, st>>>(codes, scales, nullptr, tensor_scale, Tb, N, K, What, ldo);
    note_launch();
    return cudaGetLastError();
}

}  // namespace aaac
