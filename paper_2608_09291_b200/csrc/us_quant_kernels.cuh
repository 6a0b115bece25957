// The quantiser of a chained call: per-token absmax of an fp16 activation (for the head of a chain;
// inside a chain the SpMM kernel's epilogue leaves it), and the quantisation of the activation to
// packed INT4 codes and fp16 scales, run once between two SpMM kernels.
#pragma once
#include "us_spmm_kernel.cuh"

namespace us {

// ---- per-token symmetric INT4 quantisation of an fp16 activation ------------------------------
// scale s = RN_fp16(amax / 7) (what the dequantisation multiplies by), reciprocal step
// inv = min(RN_fp16(7 / amax), 65504), code = clamp(RNE(y * inv), -8, 7) with the product exact.
__device__ __forceinline__ float requant_scale(uint32_t amax_bits)
{
    const float a = __half2float(__ushort_as_half((unsigned short)amax_bits));
    return __half2float(__float2half_rn(__fdiv_rn(a, 7.0f)));
}
__device__ __forceinline__ unsigned short requant_inverse(uint32_t amax_bits)
{
    const float a = __half2float(__ushort_as_half((unsigned short)amax_bits));
    const float inv = __fdiv_rn(7.0f, a);                 // +inf for amax = 0
    const __half h = __float2half_rn(inv);                // +inf above the fp16 range
    return (unsigned short)min((uint32_t)__half_as_ushort(h), 0x7BFFu);   // positive: bit patterns order like values
}
// eight fp16 values (four words, element e in half e) -> one word of eight INT4 codes (element e in
// nibble e): the layout of the packed INT4 input. One fused multiply-add per pair of values lands
// the product, rounded to nearest-even, in the integer bits of 1536 + q (fp16 spacing there is 1);
// the clamp to [1528, 1543] = 1536 + [-8, 7] leaves the two's-complement nibble in bits 0..3.
__device__ __forceinline__ uint32_t requant8(const uint4 h, uint32_t inv2_bits)
{
    const __half2 inv2 = *reinterpret_cast<const __half2*>(&inv2_bits);
    const __half2 magic = __floats2half2_rn(1536.f, 1536.f);
    const __half2 lo = __floats2half2_rn(1528.f, 1528.f), hi = __floats2half2_rn(1543.f, 1543.f);
    const uint32_t w[4] = {h.x, h.y, h.z, h.w};
    uint32_t v = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __half2 r = __hfma2(*reinterpret_cast<const __half2*>(&w[i]), inv2, magic);
        r = __hmin2(__hmax2(r, lo), hi);
        const uint32_t b = *reinterpret_cast<const uint32_t*>(&r);
        v |= ((b & 0xFu) | ((b >> 12) & 0xF0u)) << (8 * i);
    }
    return v;
}

// Absmax buffer of X16 (layout in us_spmm_kernel.cuh): block (bx, n) writes part bx of token n.
// Grid (P, N) with P <= kAmaxParts; all 64 token slots of every part are written (zero beyond N).
__global__ void __launch_bounds__(256) us_absmax_f16_kernel(const uint16_t* X16, int64_t ldx, int64_t K, int N,
                                                            uint32_t* amax)
{
    __shared__ uint32_t red[8];
    const int n = blockIdx.y;
    const uint16_t* row = X16 + (int64_t)n * ldx;
    uint32_t big = 0;
    const bool vec = (ldx % 8 == 0) && (reinterpret_cast<uintptr_t>(X16) % 16 == 0);
    const int64_t units = (K + 7) / 8;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (int64_t)gridDim.x * blockDim.x) {
        const int64_t k = 8 * u;
        if (vec && k + 8 <= K) {
            const uint4 h = __ldcg(reinterpret_cast<const uint4*>(row + k));
            const uint32_t w[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) big = max(big, max(w[i] & 0x7FFFu, (w[i] >> 16) & 0x7FFFu));
        } else {
            for (int e = 0; e < 8 && k + e < K; ++e) big = max(big, (uint32_t)(__ldcg(row + k + e) & 0x7FFFu));
        }
    }
    big = __reduce_max_sync(0xffffffffu, big);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = big;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) big = max(big, red[w]);
        amax[64 + 64 * blockIdx.x + n] = big;
        if (n == 0) {
            for (int t = N; t < 64; ++t) amax[64 + 64 * blockIdx.x + t] = 0;
            if (blockIdx.x == 0) amax[0] = gridDim.x;
        }
    }
}

// Xq[n][k/2] = packed INT4 codes (even k in the low nibble), x_scale[n] = the dequantisation scale as
// fp16 bits. Grid (chunks, N).
__global__ void __launch_bounds__(256) us_quantize_f16_kernel(const uint16_t* X16, int64_t ldx, int64_t K,
                                                              const uint32_t* amax, uint8_t* Xq, uint16_t* x_scale)
{
    __shared__ uint32_t am;
    const int n = blockIdx.y;
    // Launched with programmatic stream serialization: the next kernel may start its prologue now;
    // the activations and their absmax may come from the kernel before, so wait for it.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) am = 0;
    __syncthreads();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    {
        const int parts = min((int)__ldcg(amax), kAmaxParts);
        uint32_t big = 0;
        for (int pt = threadIdx.x; pt < parts; pt += blockDim.x) big = max(big, __ldcg(amax + 64 + 64 * pt + n) & 0x7FFFu);
        big = __reduce_max_sync(0xffffffffu, big);
        if ((threadIdx.x & 31) == 0 && big) atomicMax(&am, big);
    }
    __syncthreads();
    const uint16_t* row = X16 + (int64_t)n * ldx;
    uint8_t* out = Xq + (int64_t)n * ((K + 1) / 2);
    const uint32_t iv = requant_inverse(am), inv2 = iv | (iv << 16);
    if (blockIdx.x == 0 && threadIdx.x == 0 && x_scale) x_scale[n] = __half_as_ushort(__float2half_rn(requant_scale(am)));
    const bool vec = (ldx % 8 == 0) && (reinterpret_cast<uintptr_t>(X16) % 16 == 0);
    const bool vec_out = (((K + 1) / 2) % 4 == 0) && (reinterpret_cast<uintptr_t>(Xq) % 4 == 0);
    const int64_t units = (K + 7) / 8;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (int64_t)gridDim.x * blockDim.x) {
        const int64_t k = 8 * u;
        uint4 h = make_uint4(0, 0, 0, 0);
        if (vec && k + 8 <= K) {
            h = __ldcg(reinterpret_cast<const uint4*>(row + k));
        } else {
            uint32_t w[4] = {0, 0, 0, 0};
            for (int e = 0; e < 8; ++e)
                if (k + e < K) w[e >> 1] |= (uint32_t)__ldcg(row + k + e) << (16 * (e & 1));
            h = make_uint4(w[0], w[1], w[2], w[3]);
        }
        const uint32_t v = requant8(h, inv2);
        if (vec_out && k + 8 <= K) {
            *reinterpret_cast<uint32_t*>(out + k / 2) = v;
        } else {
            for (int e = 0; e < 8; e += 2)
                if (k + e < K) out[(k + e) / 2] = (uint8_t)((v >> (4 * e)) & (k + e + 1 < K ? 0xFFu : 0x0Fu));
        }
    }
}

}  // namespace us
