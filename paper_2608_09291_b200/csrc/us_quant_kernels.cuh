// Helper kernels around a chained call: per-token absmax of an fp16 activation, and its
// quantisation to packed INT4 with the step requant_step() defines (us_spmm_kernel.cuh). The SpMM
// kernel does both inside its own staging and epilogue; these serve the head of a chain and calls
// that want the codes themselves.
#pragma once
#include "us_spmm_kernel.cuh"

namespace us {

// amax[n] = max_k |X16[n][k]| (fp16 bit pattern in a 32-bit word). One CTA per (token, column chunk);
// amax must be zero on entry.
__global__ void __launch_bounds__(256) us_absmax_f16_kernel(const uint16_t* X16, int64_t ldx, int64_t K,
                                                            uint32_t* amax)
{
    const int n = blockIdx.y;
    const uint16_t* row = X16 + (int64_t)n * ldx;
    uint32_t big = 0;
    const bool vec = (ldx % 8 == 0) && (reinterpret_cast<uintptr_t>(X16) % 16 == 0);
    const int64_t units = (K + 7) / 8;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (int64_t)gridDim.x * blockDim.x) {
        const int64_t k = 8 * u;
        if (vec && k + 8 <= K) {
            const uint4 h = __ldg(reinterpret_cast<const uint4*>(row + k));
            const uint32_t w[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) big = max(big, max(w[i] & 0x7FFFu, (w[i] >> 16) & 0x7FFFu));
        } else {
            for (int e = 0; e < 8 && k + e < K; ++e) big = max(big, (uint32_t)(__ldg(row + k + e) & 0x7FFFu));
        }
    }
    big = __reduce_max_sync(0xffffffffu, big);
    if ((threadIdx.x & 31) == 0 && big) atomicMax(amax + n, big);
}

// Xq[n][k/2] = packed INT4 codes (even k in the low nibble), x_scale[n] = the step as fp16 bits.
__global__ void __launch_bounds__(256) us_quantize_f16_kernel(const uint16_t* X16, int64_t ldx, int64_t K,
                                                              const uint32_t* amax, uint8_t* Xq, uint16_t* x_scale)
{
    const int n = blockIdx.y;
    const uint16_t* row = X16 + (int64_t)n * ldx;
    uint8_t* out = Xq + (int64_t)n * ((K + 1) / 2);
    const float step = requant_step(__ldg(amax + n));
    if (blockIdx.x == 0 && threadIdx.x == 0 && x_scale) x_scale[n] = __half_as_ushort(__float2half_rn(step));
    const bool vec = (ldx % 8 == 0) && (reinterpret_cast<uintptr_t>(X16) % 16 == 0);
    const bool vec_out = (((K + 1) / 2) % 4 == 0) && (reinterpret_cast<uintptr_t>(Xq) % 4 == 0);
    const int64_t units = (K + 7) / 8;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (int64_t)gridDim.x * blockDim.x) {
        const int64_t k = 8 * u;
        uint4 h = make_uint4(0, 0, 0, 0);
        if (vec && k + 8 <= K) {
            h = __ldg(reinterpret_cast<const uint4*>(row + k));
        } else {
            uint32_t w[4] = {0, 0, 0, 0};
            for (int e = 0; e < 8; ++e)
                if (k + e < K) w[e >> 1] |= (uint32_t)__ldg(row + k + e) << (16 * (e & 1));
            h = make_uint4(w[0], w[1], w[2], w[3]);
        }
        const uint32_t v = requant8(h, step);
        if (vec_out && k + 8 <= K) {
            *reinterpret_cast<uint32_t*>(out + k / 2) = v;
        } else {
            for (int e = 0; e < 8; e += 2)
                if (k + e < K) out[(k + e) / 2] = (uint8_t)((v >> (4 * e)) & (k + e + 1 < K ? 0xFFu : 0x0Fu));
        }
    }
}

}  // namespace us
