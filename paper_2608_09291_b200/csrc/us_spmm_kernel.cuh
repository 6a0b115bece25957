// sm_100a SpMM kernel: lane-stream IE-BME weights (see us_host.h) x dense INT4 activations.
//
// Steps of the hot path (paper Alg. 2 / Sec. VI, re-designed for B200):
//   schedule   persistent CTAs, one per SM; CTA c owns tiles [cta_begin[c], cta_begin[c+1]) of
//              the segment-major tile sequence (byte balanced on the host); warps claim tiles
//              from a shared-memory counter.
//   stage W    every warp runs its own ring of STAGES slots; one cp.async.bulk per tile
//              (bitmaps + payload are one contiguous blob) completing on an mbarrier
//              (the role of the paper's double-buffered producer/consumer pipeline, Sec. VI-A).
//   stage X    the CTA expands the INT4 activations of the current K segment once into int8
//              (x16, so no per-element sign extension) in shared memory.
//   decode     bitmap -> operand fragment (the role of LSPD, Sec. VI-B): per lane and k-block
//              one mask byte indexes a 256-entry selector table; two byte-permutes deposit the
//              payload bytes of the lane's stream into the 8 fragment slots, absent positions
//              take the neutral byte 0x08. All loads hit the lane's own shared-memory bank.
//   MMA        mma.sync m16n8k32 s8: fragment rows g carry the raw payload bytes
//              (16*w_hi + (w_lo+8)), rows g+8 the low nibbles (w_lo+8); with Sx = sum_k x,
//              Y_lo = E - 8*Sx and Y_hi = (RAW - E)/16, all exact in INT32.
//   reduce     split-K partial sums go to an INT32 workspace with red.add; the warp whose
//              arrival completes a strip reads the sums, applies the optional fp16 dequant
//              epilogue, stores Y and leaves workspace and counter zeroed.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace us {

struct SpmmParams {
    const uint8_t* blob;
    const uint32_t* item_off;   // n_items + 1, units of 16 bytes
    const uint32_t* cta_begin;  // gridDim.x + 1
    const int32_t* row_order;   // Mp entries
    const uint16_t* w_scale;    // M fp16 bit patterns or nullptr
    const uint8_t* X;           // N x ceil(K/2) packed INT4
    const uint16_t* x_scale;    // N fp16 bit patterns or nullptr
    void* Y;                    // N x M int32 or fp16
    int32_t* acc;               // split-K workspace, zero between calls
    uint32_t* cnt;              // per-strip arrival counters, zero between calls
    uint32_t* err;              // device error word
    int32_t M, K, N;
    int32_t n_strips, n_segs;
    int32_t nkb, mask_rows, K_L;
    uint32_t slot_bytes;        // ring slot size (max tile blob + slack), multiple of 128
    int32_t x_fast;             // X rows are 4-byte aligned and K % 8 == 0
    int32_t fp16_out;
};

constexpr uint32_t kLutBytes = 256 * 32 * 4;
constexpr uint32_t kFill = 0x08080808u;
constexpr uint32_t kErrTimeout = 1;

// ---- selector table -------------------------------------------------------------------------
// entry(m): low 16 bits  = prmt selector for mask bits 0..3 reading the 4 bytes AT the lane's
//                          stream position (nibble j = rank of bit j, or 4 = neutral byte);
//           high 16 bits = prmt selector for mask bits 4..7 reading the 4 bytes that END at the
//                          stream position after this k-block (nibble j = 4 - c_hi + rank).
struct LutTable {
    uint32_t v[256];
};
constexpr LutTable make_lut()
{
    LutTable t{};
    for (int m = 0; m < 256; ++m) {
        uint32_t lo = 0, hi = 0;
        int rank = 0;
        for (int j = 0; j < 4; ++j) {
            uint32_t s = 4;
            if ((m >> j) & 1) s = rank++;
            lo |= s << (4 * j);
        }
        int c_hi = 0;
        for (int j = 4; j < 8; ++j) c_hi += (m >> j) & 1;
        rank = 0;
        for (int j = 4; j < 8; ++j) {
            uint32_t s = 4;
            if ((m >> j) & 1) s = 4 - c_hi + rank++;
            hi |= s << (4 * (j - 4));
        }
        t.v[m] = lo | (hi << 16);
    }
    return t;
}
__constant__ LutTable c_lut = make_lut();

// ---- PTX helpers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after ~2 s of wall time (or 2^22 polls) instead of spinning forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > 2000000000ull) break;
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                       uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- X staging: INT4 -> int8 (x16) for one K segment, plus 16 * sum_k x per token -------------
template <int NT>
__device__ __forceinline__ void stage_x(const SpmmParams& p, int sg, uint8_t* x8, int32_t* sx16,
                                        int warp, int lane, int n_warps)
{
    const int xstride = p.K_L + 32;
    const int words = p.K_L / 8;  // one word = 8 activations
    const int64_t ldx = ((int64_t)p.K + 1) / 2;
    const int64_t k0 = (int64_t)sg * p.K_L;
    for (int n = warp; n < NT * 8; n += n_warps) {
        int32_t s = 0;
        for (int wi = lane; wi < words; wi += 32) {
            const int64_t k = k0 + 8 * wi;
            uint32_t v = 0;
            if (n < p.N) {
                const uint8_t* src = p.X + (int64_t)n * ldx + k / 2;
                if (p.x_fast && k + 8 <= p.K) {
                    v = *reinterpret_cast<const uint32_t*>(src);
                } else {
                    for (int e = 0; e < 8; ++e) {
                        if (k + e < p.K) {
                            uint32_t byte = src[e >> 1];
                            v |= ((e & 1) ? (byte >> 4) : (byte & 0xF)) << (4 * e);
                        }
                    }
                }
            }
            const uint32_t te = (v << 4) & 0xF0F0F0F0u;  // 16*x for k even
            const uint32_t to = v & 0xF0F0F0F0u;         // 16*x for k odd
            uint2 o;
            o.x = prmt(te, to, 0x5140);
            o.y = prmt(te, to, 0x7362);
            *reinterpret_cast<uint2*>(x8 + n * xstride + 8 * wi) = o;
            s = __dp4a((int)te, 0x01010101, s);
            s = __dp4a((int)to, 0x01010101, s);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) sx16[n] = s;
    }
}

// ---- decode + MMA over one staged tile ---------------------------------------------------------
template <int NT>
__device__ __forceinline__ void process_tile(const uint32_t* __restrict__ slot,
                                             const uint32_t* __restrict__ lut,
                                             const uint8_t* __restrict__ x8, int xstride,
                                             int mask_rows, int lane, int (&c)[NT][4])
{
    const int g = lane >> 2, t = lane & 3;
    const uint32_t* maskp = slot + lane;
    const uint32_t* payp = slot + mask_rows * 32 + lane;
    const uint32_t* lutp = lut + lane;
    const uint8_t* xb = x8 + g * xstride + 8 * t;
    uint32_t b8 = 0;  // 8 * (byte position in the lane's payload stream)
    uint32_t d0 = 0, sel_hi = 0;

    auto finish_block = [&](int kb, uint32_t prev) {
        const uint32_t d1 = prmt(prev, kFill, sel_hi);
        const uint32_t e0 = d0 & 0x0F0F0F0Fu, e1 = d1 & 0x0F0F0F0Fu;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const uint2 b = *reinterpret_cast<const uint2*>(xb + nt * 8 * xstride + kb * 32);
            mma_s8(c[nt], d0, e0, d1, e1, b.x, b.y);
        }
    };

    for (int w = 0; w < mask_rows; ++w) {
        const uint32_t mw = maskp[w * 32];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t* q = payp + ((b8 >> 5) << 5);
            const uint32_t wm1 = *(q - 32), w0 = q[0], w1 = q[32];
            const uint32_t prev = __funnelshift_r(wm1, w0, b8);
            const uint32_t lo = __funnelshift_r(w0, w1, b8);
            if (w > 0 || i > 0) finish_block(4 * w + i - 1, prev);
            const uint32_t mb = (mw >> (8 * i)) & 0xFFu;
            const uint32_t e = lutp[mb * 32];
            d0 = prmt(lo, kFill, e);
            sel_hi = e >> 16;
            b8 += 8u * (uint32_t)__popc(mb);
        }
    }
    {
        const uint32_t* q = payp + ((b8 >> 5) << 5);
        const uint32_t prev = __funnelshift_r(*(q - 32), q[0], b8);
        finish_block(4 * mask_rows - 1, prev);
    }
}

// ---- the kernel -----------------------------------------------------------------------------
template <int NT, int STAGES>
__global__ void __launch_bounds__(512, 1) us_spmm_kernel(const SpmmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const uint32_t beg = p.cta_begin[blockIdx.x], end = p.cta_begin[blockIdx.x + 1];
    if (beg >= end) return;

    const int xstride = p.K_L + 32;
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem);
    uint8_t* x8 = smem + kLutBytes;
    int32_t* sx16 = reinterpret_cast<int32_t*>(x8 + NT * 8 * xstride);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sx16 + 64);
    uint32_t* claim = reinterpret_cast<uint32_t*>(bars + 32 * STAGES);
    uint8_t* ring0 = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(claim + 32) + 127) & ~uintptr_t(127));
    uint8_t* my_ring = ring0 + (size_t)warp * STAGES * p.slot_bytes;

    // selector table, replicated once per bank
    for (int e = warp; e < 256; e += n_warps) lut[e * 32 + lane] = c_lut.v[e];
    if (threadIdx.x == 0) *claim = beg;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(smem_u32(&bars[warp * STAGES + s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    uint32_t item[STAGES];
    uint32_t phase = 0;   // bit s = parity to wait for on stage s
    bool dead = false;    // a bounded wait ran out: stop working, keep the barriers balanced

    auto issue = [&](int s) {
        uint32_t it = 0;
        if (lane == 0) it = atomicAdd(claim, 1u);
        it = __shfl_sync(0xffffffffu, it, 0);
        item[s] = it;
        if (it < end && lane == 0) {
            const uint32_t o0 = p.item_off[it], o1 = p.item_off[it + 1];
            const uint32_t bytes = (o1 - o0) * 16u;
            const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
            // the warp's earlier generic-proxy reads of this slot are ordered before the refill
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(bar, bytes);
            bulk_g2s(smem_u32(my_ring + (size_t)s * p.slot_bytes), p.blob + (size_t)o0 * 16u, bytes, bar);
        }
    };
#pragma unroll
    for (int s = 0; s < STAGES; ++s) issue(s);

    const int sg_first = beg / p.n_strips, sg_last = (end - 1) / p.n_strips;
    int cur = 0;
    for (int sg = sg_first; sg <= sg_last; ++sg) {
        if (sg != sg_first) __syncthreads();  // everyone is done with the previous segment's X
        stage_x<NT>(p, sg, x8, sx16, warp, lane, n_warps);
        __syncthreads();

        while (!dead) {
            // the oldest claimed tile of this warp (static indexing of item[])
            uint32_t it = 0;
#pragma unroll
            for (int s = 0; s < STAGES; ++s)
                if (s == cur) it = item[s];
            if (it >= end || (int)(it / p.n_strips) != sg) break;

            const uint32_t bar = smem_u32(&bars[warp * STAGES + cur]);
            if (!mbar_wait_bounded(bar, (phase >> cur) & 1u)) {
                if (lane == 0) atomicExch(p.err, kErrTimeout);
                dead = true;
                break;
            }
            phase ^= 1u << cur;

            int c[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0;
            const uint32_t* slot = reinterpret_cast<const uint32_t*>(my_ring + (size_t)cur * p.slot_bytes);
            process_tile<NT>(slot, lut, x8, xstride, p.mask_rows, lane, c);
            __syncwarp();

            // refill this slot before the epilogue so the copy overlaps it
#pragma unroll
            for (int s = 0; s < STAGES; ++s)
                if (s == cur) issue(s);
            cur = (cur + 1 == STAGES) ? 0 : cur + 1;

            // ---- split-K reduce + finalize ----
            const int rb = (int)(it % p.n_strips);
            const int t2 = (lane & 3) * 2;
            int32_t* accp = p.acc + (size_t)rb * (NT * 128) + lane;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int n0 = nt * 8 + t2;
                const int s0 = sx16[n0] >> 4, s1 = sx16[n0 + 1] >> 4;
                const int e0 = c[nt][2] >> 4, e1 = c[nt][3] >> 4;
                const int ylo0 = e0 - 8 * s0, ylo1 = e1 - 8 * s1;           // strip row g
                const int yhi0 = (c[nt][0] - c[nt][2]) >> 8, yhi1 = (c[nt][1] - c[nt][3]) >> 8;  // row g+8
                if (p.n_segs == 1) {
                    c[nt][0] = ylo0; c[nt][1] = ylo1; c[nt][2] = yhi0; c[nt][3] = yhi1;
                } else {
                    atomicAdd(accp + nt * 128 + 0, ylo0);
                    atomicAdd(accp + nt * 128 + 32, ylo1);
                    atomicAdd(accp + nt * 128 + 64, yhi0);
                    atomicAdd(accp + nt * 128 + 96, yhi1);
                }
            }
            bool last = true;
            if (p.n_segs > 1) {
                __threadfence();
                __syncwarp();
                uint32_t old = 0;
                if (lane == 0) old = atomicAdd(p.cnt + rb, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                last = (old == (uint32_t)p.n_segs - 1);
                if (last) {
                    __threadfence();
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            c[nt][j] = __ldcg(accp + nt * 128 + j * 32);
                            __stcg(accp + nt * 128 + j * 32, 0);
                        }
                    if (lane == 0) p.cnt[rb] = 0;
                }
            }
            if (last) {
                const int g = lane >> 2;
                const int m_lo = p.row_order[rb * 16 + g], m_hi = p.row_order[rb * 16 + g + 8];
                float sw_lo = 0.f, sw_hi = 0.f;
                if (p.fp16_out) {
                    if (m_lo >= 0) sw_lo = __half2float(__ushort_as_half(p.w_scale[m_lo]));
                    if (m_hi >= 0) sw_hi = __half2float(__ushort_as_half(p.w_scale[m_hi]));
                }
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int n = nt * 8 + t2 + (j & 1);
                        const int m = (j < 2) ? m_lo : m_hi;
                        if (n >= p.N || m < 0) continue;
                        const size_t o = (size_t)n * p.M + m;
                        if (p.fp16_out) {
                            const float sx = __half2float(__ushort_as_half(p.x_scale[n]));
                            const float v = (float)c[nt][j] * ((j < 2) ? sw_lo : sw_hi) * sx;
                            reinterpret_cast<__half*>(p.Y)[o] = __float2half_rn(v);
                        } else {
                            reinterpret_cast<int32_t*>(p.Y)[o] = c[nt][j];
                        }
                    }
            }
        }
    }

    // Drain: copies this warp issued but never consumed must land before the CTA exits.
#pragma unroll
    for (int s = 0; s < STAGES; ++s) {
        if (item[s] < end) {
            const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
            if (!mbar_wait_bounded(bar, (phase >> s) & 1u) && lane == 0) atomicExch(p.err, kErrTimeout);
        }
    }
}

}  // namespace us
