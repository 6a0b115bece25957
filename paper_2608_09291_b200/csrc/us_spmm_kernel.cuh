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
    unsigned long long* timers; // optional stage timers (5 counters) or nullptr
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

// ---- decode + MMA over one staged tile -------------------------------------------------------
// CH independent decode chains walk consecutive ranges of the tile's k-blocks (chain ch starts at
// the lane-stream position given by the popcount of the mask words before its range); the chains
// only share the accumulators, so their shared-memory and permute latencies overlap.
template <int NT, int CH>
__device__ __forceinline__ void process_tile(const uint32_t* __restrict__ slot,
                                             const uint32_t* __restrict__ lut,
                                             const uint8_t* __restrict__ x8, int xstride,
                                             int mask_rows, int lane, int (&c)[NT][4])
{
    const int g = lane >> 2, t = lane & 3;
    const int rows_per = mask_rows / CH;
    const uint32_t* maskp = slot + lane;
    const uint32_t* payp = slot + mask_rows * 32 + lane;
    const uint32_t* lutp = lut + lane;
    const uint8_t* xb = x8 + g * xstride + 8 * t;
    uint32_t b8[CH];   // 8 * (byte position in the lane's payload stream), per chain
    uint32_t d0[CH], sel_hi[CH];
    b8[0] = 0;
#pragma unroll
    for (int ch = 1; ch < CH; ++ch) {
        uint32_t n = 0;
        for (int w = 0; w < rows_per; ++w) n += (uint32_t)__popc(maskp[((ch - 1) * rows_per + w) * 32]);
        b8[ch] = b8[ch - 1] + 8u * n;
    }
#pragma unroll
    for (int ch = 0; ch < CH; ++ch) d0[ch] = sel_hi[ch] = 0;

    auto finish_block = [&](int ch, int kb, uint32_t prev) {
        const uint32_t d1 = prmt(prev, kFill, sel_hi[ch]);
        const uint32_t e0 = d0[ch] & 0x0F0F0F0Fu, e1 = d1 & 0x0F0F0F0Fu;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const uint2 b = *reinterpret_cast<const uint2*>(xb + nt * 8 * xstride + kb * 32);
            mma_s8(c[nt], d0[ch], e0, d1, e1, b.x, b.y);
        }
    };

    for (int w = 0; w < rows_per; ++w) {
        uint32_t mw[CH];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) mw[ch] = maskp[(ch * rows_per + w) * 32];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int ch = 0; ch < CH; ++ch) {
                const uint32_t* q = payp + ((b8[ch] >> 5) << 5);
                const uint32_t wm1 = *(q - 32), w0 = q[0], w1 = q[32];
                const uint32_t prev = __funnelshift_r(wm1, w0, b8[ch]);
                const uint32_t lo = __funnelshift_r(w0, w1, b8[ch]);
                if (w > 0 || i > 0) finish_block(ch, 4 * (ch * rows_per + w) + i - 1, prev);
                const uint32_t mb = (mw[ch] >> (8 * i)) & 0xFFu;
                const uint32_t e = lutp[mb * 32];
                d0[ch] = prmt(lo, kFill, e);
                sel_hi[ch] = e >> 16;
                b8[ch] += 8u * (uint32_t)__popc(mb);
            }
        }
    }
#pragma unroll
    for (int ch = 0; ch < CH; ++ch) {
        const uint32_t* q = payp + ((b8[ch] >> 5) << 5);
        const uint32_t prev = __funnelshift_r(*(q - 32), q[0], b8[ch]);
        finish_block(ch, 4 * (ch + 1) * rows_per - 1, prev);
    }
}

// ---- the kernel -----------------------------------------------------------------------------
template <int NT, int STAGES, int CH>
__global__ void __launch_bounds__(512, 1) us_spmm_kernel(const SpmmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const uint32_t beg = __ldg(p.cta_begin + blockIdx.x), end = __ldg(p.cta_begin + blockIdx.x + 1);
    if (beg >= end) return;

    const int xstride = p.K_L + 32;
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem);
    uint8_t* x8 = smem + kLutBytes;
    int32_t* sx16 = reinterpret_cast<int32_t*>(x8 + NT * 8 * xstride);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sx16 + 64);
    uint8_t* ring0 = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(bars + 32 * STAGES + 16) + 127) & ~uintptr_t(127));
    uint8_t* my_ring = ring0 + (size_t)warp * STAGES * p.slot_bytes;
    const bool timing = p.timers != nullptr;
    long long t_wait = 0, t_decode = 0, t_epi = 0, t_start = timing ? clock64() : 0;

    // ---- this warp's tiles: beg + warp, beg + warp + n_warps, ... (static round robin) --------
    // Start the first copies before anything else: the barriers are private to the warp.
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(smem_u32(&bars[warp * STAGES + s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    uint32_t next_issue = beg + warp;  // next tile to start a copy for
    uint32_t next_proc = beg + warp;   // next tile to decode
    uint32_t po0 = 0, po1 = 0;         // offsets of tile next_issue (valid in lane 0)
    {
        // lanes 0..STAGES fetch the offsets of the first STAGES+1 tiles in parallel
        uint32_t o0 = 0, o1 = 0;
        const uint32_t mine = next_issue + (uint32_t)lane * (uint32_t)n_warps;
        if (lane <= STAGES && mine < end) { o0 = __ldg(p.item_off + mine); o1 = __ldg(p.item_off + mine + 1); }
#pragma unroll
        for (int s = 0; s <= STAGES; ++s) {
            const uint32_t a = __shfl_sync(0xffffffffu, o0, s), b = __shfl_sync(0xffffffffu, o1, s);
            if (s < STAGES) {
                if (next_issue < end && lane == 0) {
                    const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
                    mbar_expect_tx(bar, (b - a) * 16u);
                    bulk_g2s(smem_u32(my_ring + (size_t)s * p.slot_bytes), p.blob + (size_t)a * 16u, (b - a) * 16u, bar);
                }
                next_issue += n_warps;
            } else {
                po0 = a; po1 = b;
            }
        }
    }
    // refill slot s with tile next_issue (offsets prefetched into po0/po1), then prefetch the next
    auto refill = [&](int s) {
        if (lane == 0 && next_issue < end) {
            const uint32_t bytes = (po1 - po0) * 16u;
            const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
            // the warp's earlier generic-proxy reads of this slot are ordered before the refill
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(bar, bytes);
            bulk_g2s(smem_u32(my_ring + (size_t)s * p.slot_bytes), p.blob + (size_t)po0 * 16u, bytes, bar);
        }
        next_issue += n_warps;
        if (lane == 0 && next_issue < end) {
            po0 = __ldg(p.item_off + next_issue);
            po1 = __ldg(p.item_off + next_issue + 1);
        }
    };

    // selector table, replicated once per bank
    for (int e = warp; e < 256; e += n_warps) lut[e * 32 + lane] = c_lut.v[e];

    uint32_t phase = 0;   // bit s = parity to wait for on stage s
    bool dead = false;    // a bounded wait ran out: stop working, keep the barriers balanced
    int pend_rb = -1;     // strip whose split-K contribution is issued but not yet signalled
    const int t2 = (lane & 3) * 2;

    // store the 16 x N results of strip rb held in fragment order in v
    auto store_strip = [&](int rb, int (&v)[NT][4]) {
        const int g = lane >> 2;
        const int m_lo = __ldg(p.row_order + rb * 16 + g), m_hi = __ldg(p.row_order + rb * 16 + g + 8);
        float sw_lo = 0.f, sw_hi = 0.f;
        if (p.fp16_out) {
            if (m_lo >= 0) sw_lo = __half2float(__ushort_as_half(__ldg(p.w_scale + m_lo)));
            if (m_hi >= 0) sw_hi = __half2float(__ushort_as_half(__ldg(p.w_scale + m_hi)));
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
                    const float sx = __half2float(__ushort_as_half(__ldg(p.x_scale + n)));
                    const float r = (float)v[nt][j] * ((j < 2) ? sw_lo : sw_hi) * sx;
                    reinterpret_cast<__half*>(p.Y)[o] = __float2half_rn(r);
                } else {
                    reinterpret_cast<int32_t*>(p.Y)[o] = v[nt][j];
                }
            }
    };
    // announce one finished split-K contribution to strip rb; the last arrival finalizes it
    auto signal_strip = [&](int rb) {
        __threadfence();
        __syncwarp();
        uint32_t old = 0;
        if (lane == 0) old = atomicAdd(p.cnt + rb, 1u);
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old == (uint32_t)p.n_segs - 1) {
            __threadfence();
            int32_t* accp = p.acc + (size_t)rb * (NT * 128) + lane;
            int v[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[nt][j] = __ldcg(accp + nt * 128 + j * 32);
                    __stcg(accp + nt * 128 + j * 32, 0);
                }
            if (lane == 0) p.cnt[rb] = 0;
            store_strip(rb, v);
        }
    };

    const int sg_first = beg / p.n_strips, sg_last = (end - 1) / p.n_strips;
    int cur = 0;
    for (int sg = sg_first; sg <= sg_last; ++sg) {
        if (sg != sg_first) __syncthreads();  // everyone is done with the previous segment's X
        stage_x<NT>(p, sg, x8, sx16, warp, lane, n_warps);
        __syncthreads();
        const uint32_t seg_base = (uint32_t)sg * (uint32_t)p.n_strips;
        const uint32_t seg_end = min(end, seg_base + (uint32_t)p.n_strips);

        while (!dead && next_proc < seg_end) {
            const long long t0 = timing ? clock64() : 0;
            const uint32_t bar = smem_u32(&bars[warp * STAGES + cur]);
            if (!mbar_wait_bounded(bar, (phase >> cur) & 1u)) {
                if (lane == 0) atomicExch(p.err, kErrTimeout);
                dead = true;
                break;
            }
            phase ^= 1u << cur;
            const long long t1 = timing ? clock64() : 0;

            int c[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0;
            const uint32_t* slot = reinterpret_cast<const uint32_t*>(my_ring + (size_t)cur * p.slot_bytes);
            process_tile<NT, CH>(slot, lut, x8, xstride, p.mask_rows, lane, c);
            __syncwarp();
            const long long t2c = timing ? clock64() : 0;

            refill(cur);  // before the epilogue, so that the copy overlaps it
            cur = (cur + 1 == STAGES) ? 0 : cur + 1;

            // ---- split-K reduce + finalize ----
            const int rb = (int)(next_proc - seg_base);
            next_proc += n_warps;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int n0 = nt * 8 + t2;
                const int s0 = sx16[n0] >> 4, s1 = sx16[n0 + 1] >> 4;
                const int e0 = c[nt][2] >> 4, e1 = c[nt][3] >> 4;
                const int yhi0 = (c[nt][0] - c[nt][2]) >> 8, yhi1 = (c[nt][1] - c[nt][3]) >> 8;  // row g+8
                c[nt][0] = e0 - 8 * s0; c[nt][1] = e1 - 8 * s1;                                 // row g
                c[nt][2] = yhi0; c[nt][3] = yhi1;
            }
            if (p.n_segs == 1) {
                store_strip(rb, c);
            } else {
                // The previous tile's red.adds were issued a whole tile ago: its fence is cheap now.
                if (pend_rb >= 0) signal_strip(pend_rb);
                int32_t* accp = p.acc + (size_t)rb * (NT * 128) + lane;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int j = 0; j < 4; ++j) atomicAdd(accp + nt * 128 + j * 32, c[nt][j]);
                pend_rb = rb;
            }
            if (timing) {
                const long long t3 = clock64();
                t_wait += t1 - t0; t_decode += t2c - t1; t_epi += t3 - t2c;
            }
        }
    }
    if (pend_rb >= 0) signal_strip(pend_rb);

    // Drain: copies this warp issued but never consumed must land before the CTA exits
    // (only after a bounded wait ran out; in a normal run every issued tile was consumed).
    if (dead) {
        uint32_t it = next_proc;
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            if (it < end && it < next_issue) {
                const uint32_t bar = smem_u32(&bars[warp * STAGES + cur]);
                if (!mbar_wait_bounded(bar, (phase >> cur) & 1u) && lane == 0) atomicExch(p.err, kErrTimeout);
            }
            it += n_warps;
            cur = (cur + 1 == STAGES) ? 0 : cur + 1;
        }
    }
    if (timing && lane == 0) {
        atomicAdd(p.timers + 0, (unsigned long long)t_wait);
        atomicAdd(p.timers + 1, (unsigned long long)t_decode);
        atomicAdd(p.timers + 2, (unsigned long long)t_epi);
        atomicAdd(p.timers + 3, (unsigned long long)(clock64() - t_start));
        atomicAdd(p.timers + 4, 1ull);
    }
}

}  // namespace us
