// sm_100a SpMM kernel: lane-stream IE-BME weights (see us_host.h) x dense INT4 activations.
//
// Steps of the hot path (paper Alg. 2 / Sec. VI, re-designed for B200):
//   schedule   persistent CTAs, one per SM. The K segments are grouped into K ranges of G
//              segments whose activations fit in shared memory; tiles are processed in the
//              order (K range, strip, segment) and CTA c owns positions [cta_begin[c],
//              cta_begin[c+1]) of that sequence (byte balanced on the host). Warps claim
//              tiles from a shared-memory counter, one tile ahead of the copy they issue.
//   stage W    every warp runs its own ring of STAGES slots; one cp.async.bulk per tile
//              (bitmaps + payload are one contiguous blob) completing on an mbarrier
//              (the role of the paper's double-buffered producer/consumer pipeline, Sec. VI-A).
//   stage X    the CTA expands the INT4 activations of the current K range once into int8
//              (x16, so no per-element sign extension) in shared memory.
//   decode     bitmap -> operand fragment (the role of LSPD, Sec. VI-B): per lane and k-block
//              one mask byte indexes a 256-entry selector table; two byte-permutes deposit the
//              payload bytes of the lane's stream into the 8 fragment slots, absent positions
//              take the neutral byte 0x08. All loads hit the lane's own shared-memory bank.
//              Folded tiles (C_A = 2): one mask byte serves two k-blocks whose payload bytes sit at the
//              same position of two streams; INT2 weights: one stream whose bytes are split into two
//              nibbles after the gather (process_tile<.., CA, W2>).
//   MMA        mma.sync m16n8k32 s8: fragment rows g carry the raw payload bytes
//              (16*w_hi + (w_lo+8)), rows g+8 the low nibbles (w_lo+8); with Sx = sum_k x,
//              Y_lo = E - 8*Sx and Y_hi = (RAW - E)/16, all exact in INT32.
//   reduce     (local mode) tiles of one strip are summed in a shared-memory accumulator; the
//              warp that adds the CTA's last tile of a strip flushes it: straight to Y when the
//              CTA saw every segment of the strip, else into the global INT32 workspace.
//              (direct mode, used when a CTA would touch too many strips) every tile goes to
//              the global workspace with red.add. In both, the arrival that completes a strip
//              reads the sums, applies the optional fp16 dequant epilogue, stores Y and leaves
//              workspace and counter zeroed.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

namespace us {

constexpr int kMaxCtas = 192;   // persistent CTAs (one per SM) the schedule can describe

struct SpmmParams {
    const uint8_t* blob;
    const uint32_t* item_off;   // n_items + 1, units of 16 bytes
    const int32_t* row_order;   // Mp entries
    const uint16_t* w_scale;    // M fp16 bit patterns or nullptr
    const uint8_t* X;           // N x ceil(K/2) packed INT4
    const uint16_t* x_scale;    // N fp16 bit patterns or nullptr
    void* Y;                    // N x M int32 or fp16
    int32_t* acc;               // split-K workspace, zero between calls
    uint32_t* cnt;              // per-strip arrival counters, zero between calls
    uint32_t* err;              // device error word
    unsigned long long* timers; // optional stage timers (9 counters) or nullptr
    int32_t M, K, N;
    int32_t n_strips, n_segs;
    int32_t G;                  // segments per K range
    int32_t run_len;            // consecutive positions a warp claims at a time
    unsigned long long mg_g, mg_glast, mg_krs;  // floor(2^40/d)+1 for d = G, the last range's
                                                // segment count, n_strips * G
    int32_t s_local;            // local mode: strips a CTA may hold in shared memory (0 = direct mode)
    int32_t lut_rep;            // copies of the selector table in shared memory (8 or 32)
    int32_t mask_rows, K_L;     // mask words per lane and tile; tile width
    int32_t w2;                 // INT2 weights (the W2 kernel instantiations)
    int32_t fold_kb;            // C_A = 2: k-blocks per column area (a mask bit also covers the column that many
                                // k-blocks further on); 0 for C_A = 1
    uint32_t slot_bytes;        // ring slot size (max tile blob + slack), multiple of 128
    int32_t x_fast;             // 2: K % 32 == 0 (16-byte loads); 1: K % 8 == 0 (4-byte loads); 0: bytes
    int32_t fp16_out;
    // Chained call: the epilogue leaves the per-token absmax of the fp16 outputs of rows
    // [amax_m0, amax_m1) in an absmax buffer (layout below) for the quantiser of the next call.
    uint32_t* y_amax;           // or nullptr
    int32_t amax_m0, amax_m1;
    uint32_t wait_ns_hi;        // bounded waits give up after this many ns >> 10
    uint32_t withhold;          // test hook: position whose copy is never issued (~0u = none)
    // CTA c owns positions [cta_begin[c], cta_begin[c+1]) of the (K range, strip, segment) order.
    // Kept in the kernel parameters: the schedule is known without a global-memory round trip.
    uint32_t cta_begin[kMaxCtas + 1];
};

constexpr int kLutRepMax = 32;   // copies of the selector table: lane l reads copy l % kLutRep. Eight copies
                             // cost ~0.4 extra wavefronts per lookup (lanes sharing a copy collide only
                             // when their entries fall in the same bank) and free 24 KB for more warps.
constexpr uint32_t kLutScratchBytes = 256 * 4;   // one unreplicated copy, built first
constexpr uint32_t kFill = 0x08080808u;      // INT4 payload byte of a cleared mask bit: w_hi = 0, w_lo + 8 = 8
constexpr uint32_t kFillW2 = 0xAAAAAAAAu;    // INT2 payload byte of a cleared mask bit: four fields of 0 + 2
constexpr uint32_t kErrTimeout = 1;
constexpr int kNoRow = -2;        // "row ids not loaded yet" marker (-1 is a padding row)
constexpr int kClaimWords = 96;   // shared-memory words of the claim counter and its neighbours
constexpr int kOffTable = 256;   // tile offsets of a CTA kept in shared memory (start, end pairs)

// ---- selector table -------------------------------------------------------------------------
// entry(m): low 16 bits  = prmt selector for mask bits 0..3 reading the 4 bytes AT the lane's
//                          stream position (nibble j = rank of bit j, or 4 = neutral byte);
//           high 16 bits = prmt selector for mask bits 4..7 reading the 4 bytes that END at the
//                          stream position after this k-block (nibble j = 4 - c_hi + rank).
__host__ __device__ constexpr uint32_t lut_entry(int m)
{
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
    return lo | (hi << 16);
}

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
// The same with a suspend-time hint: the thread sleeps in hardware (taking no issue slots from the
// decoding warps) until the phase completes or about `ns` nanoseconds have passed.
__device__ __forceinline__ bool mbar_try_wait_sleep(uint32_t bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after limit_hi << 10 ns of wall time (~2 s unless a test shortens it)
// instead of spinning forever. Between checks of the clock the thread sleeps on the barrier.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit_hi)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    const uint32_t nap = limit_hi < 64u ? 1000u : 20000u;   // ns per sleep
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (mbar_try_wait_sleep(bar, parity, nap)) return true;
        if (((global_timer_ns() - t0) >> 10) > limit_hi) break;
    }
    return false;
}
// The weights are read once per call: their lines are marked evict-first in L2, so that they do not
// push out what is reused (the activations every CTA reads, the split-K workspace).
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
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

// ---- shared-memory access by 32-bit address ---------------------------------------------------
__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
// load at a compile-time byte offset from a: the offset goes into the instruction's immediate field
// instead of costing an integer add per load
template <int OFF>
__device__ __forceinline__ uint32_t lds32_at(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}

// ---- X staging: INT4 -> int8 (x16) for one K range, plus 16 * sum_k x per (segment, token) -----
// expands 8 packed activations (one 32-bit word) into two words of int8 (x16) and adds 16 * their sum
__device__ __forceinline__ uint2 expand8(uint32_t v, int32_t& s)
{
    const uint32_t te = (v << 4) & 0xF0F0F0F0u;  // 16*x for k even
    const uint32_t to = v & 0xF0F0F0F0u;         // 16*x for k odd
    s = __dp4a((int)te, 0x01010101, s);
    s = __dp4a((int)to, 0x01010101, s);
    return make_uint2(prmt(te, to, 0x5140), prmt(te, to, 0x7362));
}

// Packed staging (XP): the same 8 activations as one word q whose even nibbles are k 0..3 and odd
// nibbles k 4..7, so that the decode loop gets its two B-fragment words (x16, as int8) with
// (q << 4) & 0xF0F0F0F0 and q & 0xF0F0F0F0. Half the shared memory of the int8 form for three more
// integer instructions per n-tile and k-block.
__device__ __forceinline__ uint32_t pack8(uint32_t v, int32_t& s)
{
    const uint2 t = expand8(v, s);
    return (t.x >> 4) | t.y;
}

// sx16 must be zero on entry (the caller clears it and synchronises).
// Units below `first_unit` (of the 16-byte path) were already staged by the caller.
template <int NT, bool XP>
__device__ __forceinline__ void stage_x(const SpmmParams& p, int seg0, int n_seg, uint8_t* x8,
                                        int xstride, int32_t* sx16, int first_unit)
{
    const int64_t ldx = ((int64_t)p.K + 1) / 2;
    const int rows = NT * 8;
    if (p.x_fast == 2) {
        // 16-byte units (32 activations); all loads of a batch are issued before any is used
        const int upr = p.K_L / 32;                 // units per (segment, token)
        const int total = rows * n_seg * upr;
        constexpr int kBatch = 4;
        for (int u0 = first_unit + threadIdx.x; u0 < total; u0 += kBatch * blockDim.x) {
            uint4 v[kBatch];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int u = u0 + b * blockDim.x;
                v[b] = make_uint4(0, 0, 0, 0);
                if (u < total) {
                    const int pi = u / upr, q = u - pi * upr;
                    const int sgl = pi / rows, n = pi - sgl * rows;
                    const int64_t k = (int64_t)(seg0 + sgl) * p.K_L + 32 * q;
                    if (n < p.N && k < p.K)
                        v[b] = __ldg(reinterpret_cast<const uint4*>(p.X + (int64_t)n * ldx + k / 2));
                }
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int u = u0 + b * blockDim.x;
                if (u < total) {
                    const int pi = u / upr, q = u - pi * upr;
                    const int sgl = pi / rows, n = pi - sgl * rows;
                    int32_t s = 0;
                    if (XP) {
                        uint4 pk;
                        pk.x = pack8(v[b].x, s); pk.y = pack8(v[b].y, s);
                        pk.z = pack8(v[b].z, s); pk.w = pack8(v[b].w, s);
                        *reinterpret_cast<uint4*>(x8 + n * xstride + (sgl * p.K_L + 32 * q) / 2) = pk;
                    } else {
                        uint4 lo, hi;
                        uint2 t;
                        t = expand8(v[b].x, s); lo.x = t.x; lo.y = t.y;
                        t = expand8(v[b].y, s); lo.z = t.x; lo.w = t.y;
                        t = expand8(v[b].z, s); hi.x = t.x; hi.y = t.y;
                        t = expand8(v[b].w, s); hi.z = t.x; hi.w = t.y;
                        uint4* dst = reinterpret_cast<uint4*>(x8 + n * xstride + sgl * p.K_L + 32 * q);
                        dst[0] = lo; dst[1] = hi;
                    }
                    if (s) atomicAdd(sx16 + pi, s);
                }
            }
        }
        return;
    }
    // general path: 8 activations at a time, any K and alignment
    const int wpr = p.K_L / 8;
    const int total = rows * n_seg * wpr;
    for (int u = threadIdx.x; u < total; u += blockDim.x) {
        const int pi = u / wpr, wi = u - pi * wpr;
        const int sgl = pi / rows, n = pi - sgl * rows;
        const int64_t k = (int64_t)(seg0 + sgl) * p.K_L + 8 * wi;
        uint32_t v = 0;
        if (n < p.N) {
            const uint8_t* src = p.X + (int64_t)n * ldx + k / 2;
            if (p.x_fast == 1 && k + 8 <= p.K) {
                v = __ldg(reinterpret_cast<const uint32_t*>(src));
            } else {
                for (int e = 0; e < 8; ++e) {
                    if (k + e < p.K) {
                        uint32_t byte = src[e >> 1];
                        v |= ((e & 1) ? (byte >> 4) : (byte & 0xF)) << (4 * e);
                    }
                }
            }
        }
        int32_t s = 0;
        if (XP) *reinterpret_cast<uint32_t*>(x8 + n * xstride + (sgl * p.K_L + 8 * wi) / 2) = pack8(v, s);
        else *reinterpret_cast<uint2*>(x8 + n * xstride + sgl * p.K_L + 8 * wi) = expand8(v, s);
        if (s) atomicAdd(sx16 + pi, s);
    }
}

// ---- absmax buffer of a chained call -----------------------------------------------------------
// kAmaxWords 32-bit words: word 0 = P, the number of parts; part p < P holds, for token n < 64, the
// fp16 bit pattern of a partial max |y| at word 64 + 64 * p + n. The absmax of a token is the largest
// of its P words. Every producer writes all of its parts (one per CTA) with plain stores, so the
// buffer needs no clearing and no atomics.
constexpr int kAmaxParts = kMaxCtas;
constexpr int kAmaxWords = 64 * (1 + kAmaxParts);

// Store the 16 x N results held in fragment order in v: fragment rows g -> original row m_lo,
// rows g + 8 -> m_hi (negative = padding row), with the optional fp16 dequantisation.
struct StoreCtx {   // what the store needs, by value (the full parameter block is large)
    void* Y;
    const uint16_t* w_scale;
    const uint16_t* x_scale;
    int32_t* acc;
    uint32_t* cnt;
    int32_t M, N, fp16_out;
    uint32_t* amax_s;           // shared-memory per-token absmax of the stored fp16 values, or nullptr
    int32_t amax_m0, amax_m1;
};
// Scales fetched ahead of the store (fp16 output): the two weight scales of a lane's rows of one
// strip, and (small N only) the activation scales of the lane's tokens.
template <int NT>
struct ScalePre {
    static constexpr bool kSx = NT <= 2;
    int rb = -1;                 // strip the weight scales belong to (-1 = none)
    // raw fp16 bit patterns: converting at the point of use keeps the loads in flight meanwhile
    unsigned short sw_lo = 0, sw_hi = 0;
    bool have_sx = false;
    unsigned short sx[kSx ? NT : 1][2];
};
// AM: also track the per-token absmax of the stored fp16 values (chained calls).
template <int NT, bool AM>
__device__ __forceinline__ void store_rows(const StoreCtx p, const int (&v)[NT][4], int lane, int m_lo, int m_hi,
                                           const ScalePre<NT>* pre = nullptr, int rb = -2)
{
    const int t2 = (lane & 3) * 2;
    float sw_lo = 0.f, sw_hi = 0.f;
    if (p.fp16_out) {
        if (pre && pre->rb == rb) {
            sw_lo = __half2float(__ushort_as_half(pre->sw_lo));
            sw_hi = __half2float(__ushort_as_half(pre->sw_hi));
        } else {
            if (m_lo >= 0) sw_lo = __half2float(__ushort_as_half(__ldg(p.w_scale + m_lo)));
            if (m_hi >= 0) sw_hi = __half2float(__ushort_as_half(__ldg(p.w_scale + m_hi)));
        }
    }
    constexpr bool track = AM;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        uint32_t big[2] = {0u, 0u};   // absmax (fp16 bits) of this lane's stored values of tokens t2, t2 + 1
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = nt * 8 + t2 + (j & 1);
            const int m = (j < 2) ? m_lo : m_hi;
            if (n >= p.N || m < 0) continue;
            const size_t o = (size_t)n * p.M + m;
            if (p.fp16_out) {
                float sx;
                if (ScalePre<NT>::kSx && pre && pre->have_sx) sx = __half2float(__ushort_as_half(pre->sx[ScalePre<NT>::kSx ? nt : 0][j & 1]));
                else sx = __half2float(__ushort_as_half(__ldg(p.x_scale + n)));
                const float r = (float)v[nt][j] * ((j < 2) ? sw_lo : sw_hi) * sx;
                const __half h = __float2half_rn(r);
                reinterpret_cast<__half*>(p.Y)[o] = h;
                if (track && m >= p.amax_m0 && m < p.amax_m1) big[j & 1] = max(big[j & 1], (uint32_t)(__half_as_ushort(h) & 0x7FFFu));
            } else {
                reinterpret_cast<int32_t*>(p.Y)[o] = v[nt][j];
            }
        }
        if (track) {   // warp-uniform: the eight lanes holding a token combine, one of them publishes
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                uint32_t b = big[jj];
                b = max(b, __shfl_xor_sync(0xffffffffu, b, 4));
                b = max(b, __shfl_xor_sync(0xffffffffu, b, 8));
                b = max(b, __shfl_xor_sync(0xffffffffu, b, 16));
                if (lane < 4 && b) atomicMax(p.amax_s + nt * 8 + t2 + jj, b);
            }
        }
    }
}

// ---- decode + MMA over one staged tile -------------------------------------------------------
// One mask word = four k-blocks of the lane. The stream positions of all four (and of the next
// word's first) follow from the mask word alone, so every shared-memory load of the word is
// issued before any is used. Block i takes its first four fragment bytes from the window that
// STARTS at pos[i] and its last four from the window that ENDS at pos[i+1]; the window at
// pos[4] is carried to the next word, so each word is self-contained (no peeled first or last).
// All addresses are 32-bit shared-memory addresses: slot_a = the staged tile, lut_a = selector
// table + 4*lane, xb_a = this lane's first B-fragment of the tile's segment.
// XP: X is staged packed (one word per lane, k-block and n-tile) instead of as int8 (two words).
// CA = column areas of the format: with CA = 2 one mask byte serves two k-blocks (kb and kb + fold_kb);
// their payload bytes sit at the same position of two streams whose 128-byte rows alternate, so the
// positions, the table entry and all address arithmetic are shared and only the window loads, the
// shifts, the permutes and the MMA are done twice.
// W2 (with CA = 2): INT2 weights. The byte of a set mask bit holds the bit's four 2-bit values (each + 2): low
// nibble = column area 0 (bits 1:0 row g, 3:2 row g + 8), high nibble = column area 1. One stream, gathered as
// for CA = 1, then split: fragment rows g take the nibble 4 * (w_hi + 2) + (w_lo + 2), rows g + 8 its low two
// bits w_lo + 2; with S = sum of x over the tile's columns, Y_lo = E - 2 S and Y_hi = (RAW - E) / 4 - 2 S.
// DP (N = 1 only; NT = 1, CA = 1, plain X): no MMA. xb_a then addresses token 0's activations at this lane's own
// eight columns, and the lane accumulates its part of the two sums with four dp4a per k-block: c[0][0] = RAW,
// c[0][2] = E. The caller adds the four lanes of a row group. Measured against the MMA at N = 1 (which wastes
// seven of its eight token columns): 2-3 % faster on every shape.
template <int NT, bool XP, int CA, bool W2 = false, bool DP = false>
__device__ __forceinline__ void process_tile(uint32_t slot_a, uint32_t lut_a, uint32_t lut_stride,
                                             uint32_t xb_a, int xstride, int mask_rows, int lane,
                                             int (&c)[NT][4], uint32_t x_fold)
{
    const uint32_t mask_a = slot_a + 4u * lane;
    const uint32_t pay_a = slot_a + 128u * mask_rows + 4u * lane;
    constexpr bool kPreX = NT <= 2 && CA == 1;   // small N: fetch the X fragments together with the windows
    constexpr uint32_t kXStep = XP ? 16u : 32u;   // bytes of a token's row per k-block
    constexpr int SR = W2 ? 1 : CA;               // payload streams per lane
    constexpr int kRow = 128 * SR;                // bytes from one payload row of a stream to its next
    auto ldx = [&](uint32_t a) -> uint2 {         // the lane's two B-fragment words at address a
        if (XP) {
            const uint32_t q = lds32(a);
            return make_uint2((q * 16u) & 0xF0F0F0F0u, q & 0xF0F0F0F0u);
        }
        return lds64(a);
    };
    uint32_t b8 = 0;                                     // 8 * (byte position in the lane's payload stream)
    uint32_t cw0[SR], cw1[SR];                           // carried window: the words at / after the position
#pragma unroll
    for (int ca = 0; ca < SR; ++ca) { cw0[ca] = lds32(pay_a + 128u * ca); cw1[ca] = lds32(pay_a + kRow + 128u * ca); }
    const uint32_t xb_fold_a = xb_a + x_fold;            // X fragments of the second column area
    for (int w = 0; w < mask_rows; ++w) {
        uint32_t pos[5], wm1[SR][4], w0[SR][4], w1[SR][4], e[4];
        uint2 xf[4][kPreX ? NT : 1];
        const uint32_t mw = lds32(mask_a + 128u * w);
        pos[0] = b8;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t cum = (i == 3) ? mw : (mw & ((1u << (8 * i + 8)) - 1u));
            pos[i + 1] = b8 + 8u * (uint32_t)__popc(cum);
            e[i] = lut_a + prmt(mw, 0u, 0x4440u + i) * lut_stride;   // address of the table entry
        }
        b8 = pos[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a = pay_a + (pos[i + 1] >> 5) * (uint32_t)kRow;   // window at the block's END
            wm1[0][i] = lds32_at<-kRow>(a);
            w0[0][i] = lds32_at<0>(a);
            w1[0][i] = lds32_at<kRow>(a);
            if (SR == 2) {
                wm1[SR - 1][i] = lds32_at<128 - kRow>(a);
                w0[SR - 1][i] = lds32_at<128>(a);
                w1[SR - 1][i] = lds32_at<128 + kRow>(a);
            }
            e[i] = lds32(e[i]);
            if (kPreX) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) xf[i][nt] = ldx(xb_a + kXStep * (4 * w + i) + nt * 8 * xstride);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (W2) {
                const uint32_t s0 = (i == 0) ? cw0[0] : w0[0][i - 1];
                const uint32_t s1 = (i == 0) ? cw1[0] : w1[0][i - 1];
                const uint32_t lo = __funnelshift_r(s0, s1, pos[i]);
                const uint32_t prev = __funnelshift_r(wm1[0][i], w0[0][i], pos[i + 1]);
                const uint32_t g0 = prmt(lo, kFillW2, e[i]);
                const uint32_t g1 = prmt(prev, kFillW2, e[i] >> 16);
#pragma unroll
                for (int ca = 0; ca < 2; ++ca) {
                    const uint32_t d0 = (ca ? g0 >> 4 : g0) & 0x0F0F0F0Fu, d1 = (ca ? g1 >> 4 : g1) & 0x0F0F0F0Fu;
                    const uint32_t e0 = d0 & 0x03030303u, e1 = d1 & 0x03030303u;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint2 b = ldx((ca ? xb_fold_a : xb_a) + kXStep * (4 * w + i) + nt * 8 * xstride);
                        mma_s8(c[nt], d0, e0, d1, e1, b.x, b.y);
                    }
                }
            } else {
#pragma unroll
            for (int ca = 0; ca < CA; ++ca) {
                // first four bytes: the window starting at pos[i] (carried, or the previous block's)
                const uint32_t s0 = (i == 0) ? cw0[ca] : w0[ca][i - 1];
                const uint32_t s1 = (i == 0) ? cw1[ca] : w1[ca][i - 1];
                const uint32_t lo = __funnelshift_r(s0, s1, pos[i]);
                const uint32_t prev = __funnelshift_r(wm1[ca][i], w0[ca][i], pos[i + 1]);
                const uint32_t d0 = prmt(lo, kFill, e[i]);
                const uint32_t d1 = prmt(prev, kFill, e[i] >> 16);
                const uint32_t e0 = d0 & 0x0F0F0F0Fu, e1 = d1 & 0x0F0F0F0Fu;
                if (DP) {
                    const uint2 b = kPreX ? xf[i][0] : ldx(xb_a + kXStep * (4 * w + i));
                    c[0][0] = __dp4a((int)d0, (int)b.x, c[0][0]); c[0][0] = __dp4a((int)d1, (int)b.y, c[0][0]);
                    c[0][2] = __dp4a((int)e0, (int)b.x, c[0][2]); c[0][2] = __dp4a((int)e1, (int)b.y, c[0][2]);
                } else {
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint2 b = kPreX ? xf[i][nt] : ldx((ca ? xb_fold_a : xb_a) + kXStep * (4 * w + i) + nt * 8 * xstride);
                        mma_s8(c[nt], d0, e0, d1, e1, b.x, b.y);
                    }
                }
            }
            }
        }
#pragma unroll
        for (int ca = 0; ca < SR; ++ca) { cw0[ca] = w0[ca][3]; cw1[ca] = w1[ca][3]; }
    }
}

// Last arrival of a strip in the global workspace: read the sums, leave workspace and counter
// zeroed, dequantise and store. Kept out of line: it runs once per strip at most, and the decode
// loop's code should stay small enough for the instruction cache.
template <int NT, bool AM>
__device__ __noinline__ void finalize_strip(const StoreCtx p, int rb, int lane, int m_lo, int m_hi)
{
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
    store_rows<NT, AM>(p, v, lane, m_lo, m_hi);
}

// ---- the kernel -----------------------------------------------------------------------------
// exact floor(u / d) for u < 2^24, d < 2^16, with m = floor(2^40 / d) + 1 precomputed on the host
__device__ __forceinline__ uint32_t fdiv(uint32_t u, unsigned long long m)
{
    return (uint32_t)(((unsigned long long)u * m) >> 40);
}

// Stage-timer buffer (unsigned long long words), written by the TIMED build: one record of kWarpRec
// words per (CTA, warp) -- [0] valid, [1] wait, [2] decode, [3] epilogue, [4] lifetime, [5] cycles
// before the first tile, [6] start ns, [7] activations staged ns, [8] end ns, [9..12] prologue
// checkpoints (cycles: range known, copies issued, table done, X staged), [13] ns past the
// dependency wait.
constexpr int kWarpRec = 16, kMaxWarpsPerCta = 24;
constexpr int kTimerWords = kWarpRec * kMaxWarpsPerCta * kMaxCtas;

// LA = local mode (shared-memory strip accumulators), else direct mode.
// TIMED = record the diagnostic stage timers (a separate instantiation, so that the production
// kernel carries none of their clock reads and branches).
// AM = chained call that leaves the per-token absmax of its fp16 output (separate too: the plain
// fp16 store measured 2.5 % slower with the tracking compiled in behind a run-time flag).
// CA = column areas of the weight format (2: folded tiles).
// W2 = INT2 weights (folded format only). DP = dp4a instead of the MMA: the N = 1 kernels of the default format.
template <int NT, int STAGES, bool LA, bool TIMED, bool XP = false, bool AM = false, int CA = 1, bool W2 = false,
          bool DP = false>
// (N <= 8 kernels are compiled for up to 20 warps: 80 registers instead of 90, which lets 12 instead of 10 warps of
// two half-SM CTAs share an SM; more than 16 warps per full-SM CTA were measured and do not pay.)
__global__ void __launch_bounds__((NT == 1 && CA == 1) ? 640 : 512, 1) us_spmm_kernel(const SpmmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    constexpr bool timing = TIMED;
    long long t_wait = 0, t_decode = 0, t_epi = 0, t_start = timing ? clock64() : 0, t_first = 0;
    long long dbg[4] = {0, 0, 0, 0};   // prologue checkpoints (cycles since t_start)
    const unsigned long long g_start = timing ? global_timer_ns() : 0;

    // ---- shared-memory carve-up (mirrored by plan_launch on the host) --------------------------
    // bytes of one token's row of staged X: int8, or packed (XP); the pad keeps the 8 tokens of an
    // n-tile on different banks
    const int xstride = XP ? p.G * p.K_L / 2 + 16 : p.G * p.K_L + 32;
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem);                       // [256][lut_rep]
    uint32_t* lut1 = lut + 256 * p.lut_rep;                                  // [256] built first
    uint8_t* x8 = reinterpret_cast<uint8_t*>(lut1 + 256);
    int32_t* sx16 = reinterpret_cast<int32_t*>(x8 + NT * 8 * xstride);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sx16 + p.G * NT * 8);
    uint32_t* claim = reinterpret_cast<uint32_t*>(bars + 32 * STAGES);
    // claim[0] = the tile counter, claim[1] = warps that have finished, claim[32 ..] = per-token absmax
    // of the stored outputs (chained calls)
    uint32_t* amax_s = claim + 32;
    int32_t* acc_l = reinterpret_cast<int32_t*>(claim + kClaimWords);      // [s_local][NT*128]
    uint32_t* cnt_l = reinterpret_cast<uint32_t*>(acc_l + p.s_local * NT * 128);  // [s_local]
    uint32_t* off_s = cnt_l + p.s_local;                                    // [kOffTable][2]
    uint8_t* ring0 = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(off_s + 2 * kOffTable) + 127) & ~uintptr_t(127));
    uint8_t* my_ring = ring0 + (size_t)warp * STAGES * p.slot_bytes;

    const uint32_t beg = p.cta_begin[blockIdx.x], end = p.cta_begin[blockIdx.x + 1];
    const uint64_t w_policy = l2_evict_first_policy();
    // Programmatic dependent launch: let the next kernel of the stream start its own prologue
    // (parameter fetch, offsets, first weight tiles) while this one is still working.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (beg >= end) {   // no work: a chained call still owes its part of the absmax buffer
        if (AM && threadIdx.x < 64) {
            asm volatile("griddepcontrol.wait;" ::: "memory");   // the buffer may still be read by the kernel before
            p.y_amax[64 + 64 * blockIdx.x + threadIdx.x] = 0;
            if (blockIdx.x == 0 && threadIdx.x == 0) p.y_amax[0] = gridDim.x;
        }
        return;
    }
    if (timing) dbg[0] = clock64() - t_start;

    // position u of the processing order -> K range, strip, segment within the range, tile index
    const uint32_t kr_stride = (uint32_t)p.n_strips * (uint32_t)p.G;
    const int n_kr = (p.n_segs + p.G - 1) / p.G;
    const int g_last = p.n_segs - (n_kr - 1) * p.G;
    auto tile_of = [&](uint32_t u, int& kr, int& rb, int& sgl) -> uint32_t {
        kr = (n_kr == 1) ? 0 : (int)fdiv(u, p.mg_krs);
        const uint32_t q = u - (uint32_t)kr * kr_stride;
        const bool lastr = (kr == n_kr - 1);
        const uint32_t g_kr = lastr ? (uint32_t)g_last : (uint32_t)p.G;
        rb = (int)fdiv(q, lastr ? p.mg_glast : p.mg_g);
        sgl = (int)(q - (uint32_t)rb * g_kr);
        return (uint32_t)rb * (uint32_t)p.n_segs + (uint32_t)(kr * p.G + sgl);
    };

    // tile index of position u; with a single K range the two orders coincide
    auto tile_index = [&](uint32_t u) -> uint32_t {
        if (n_kr == 1) return u;
        int kr, rb, sgl;
        return tile_of(u, kr, rb, sgl);
    };

    // ---- tile queue of this warp: runs of R consecutive positions --------------------------------
    // The first runs are fixed (run w, w + n_warps, ...: enough to fill the ring and one ahead);
    // later runs are claimed from the CTA's counter. A run mostly stays inside one strip, so its
    // partial sums are carried in registers and flushed once.
    const uint32_t R = (uint32_t)p.run_len;
    const int n_static = (STAGES + 1 + (int)R - 1) / (int)R;   // fixed runs per warp
    auto static_pos = [&](int k) -> uint32_t {                 // k-th position of the fixed sequence
        const uint32_t j = (uint32_t)k / R, i = (uint32_t)k - j * R;
        return beg + ((uint32_t)warp + j * (uint32_t)n_warps) * R + i;
    };
    uint32_t run_next = 0, run_end = 0;   // the run being handed out (after the fixed positions)
    int static_k = STAGES + 1;            // fixed positions already handed out
    // (a CTA whose fixed positions already cover its whole range never touches the counter)
    const bool all_static = beg + (uint32_t)n_static * (uint32_t)n_warps * R >= end;
    auto next_pos = [&]() -> uint32_t {
        if (static_k < n_static * (int)R) return static_pos(static_k++);
        if (all_static) return end;
        if (run_next == run_end) {
            // Guided chunks: as long as every warp can still get a run of R (a whole strip's
            // segments when R = G: its sums never leave the registers), hand out R; towards the end
            // of the CTA's range halve the runs so that the warps finish together.
            uint32_t b = 0, n = 0;
            if (lane == 0) {
                const uint32_t seen = *(volatile uint32_t*)claim;
                const uint32_t left = seen < end ? end - seen : 0u;
                n = R;
                while (n > 1u && n * (uint32_t)n_warps > left) n >>= 1;
                b = atomicAdd(claim, n);
            }
            run_next = __shfl_sync(0xffffffffu, b, 0);
            run_end = run_next + __shfl_sync(0xffffffffu, n, 0);
        }
        return run_next++;
    };

    // ---- start the first copies: the barriers are private to the warp ---------------------------
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(smem_u32(&bars[warp * STAGES + s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    uint32_t item[STAGES];        // position u held (or awaited) by each ring slot
    uint32_t ahead;               // next position, whose offsets are already being fetched
    uint32_t po0 = 0, po1 = 0;    // its offsets (valid in lane 0)
    int pre_rb = -1, pre_mlo = -1, pre_mhi = -1;   // fp16 output: rows of the warp's first strip
    // (Only the N <= 16 kernels fetch scales ahead: the wider ones have no registers to spare --
    // measured at N = 64 on a 28672 x 8192 matrix: 102 us with this code compiled in, 87 us without.)
    constexpr bool kPreScales = NT <= 2;
    if (kPreScales && p.fp16_out && static_pos(0) < end) {
        int kr0, sg0;
        tile_of(static_pos(0), kr0, pre_rb, sg0);
        pre_mlo = __ldg(p.row_order + pre_rb * 16 + (lane >> 2));
        pre_mhi = __ldg(p.row_order + pre_rb * 16 + (lane >> 2) + 8);
    }
    {
        // lanes 0..STAGES fetch the offsets of the first STAGES+1 positions in parallel
        const uint32_t mine = static_pos(lane <= STAGES ? lane : 0);
        uint32_t o0 = 0, o1 = 0;
        if (lane <= STAGES && mine < end) {
            const uint32_t t = tile_index(mine);
            o0 = __ldg(p.item_off + t); o1 = __ldg(p.item_off + t + 1);
        }
        // meanwhile the CTA fetches the offsets of its first kOffTable positions into shared
        // memory (visible after the first __syncthreads); later refills never wait on DRAM
        for (int i = threadIdx.x; i < kOffTable; i += blockDim.x) {
            const uint32_t u = beg + (uint32_t)i;
            if (u < end) {
                const uint32_t t = tile_index(u);
                off_s[2 * i] = __ldg(p.item_off + t);
                off_s[2 * i + 1] = __ldg(p.item_off + t + 1);
            }
        }
        // (built here: its arithmetic overlaps the offset loads issued just above)
        // Selector table: every thread computes one entry (pure register arithmetic: no memory
        // round trip in the prologue); the copies are written after the next CTA barrier.
        for (int e = threadIdx.x; e < 256; e += blockDim.x) lut1[e] = lut_entry(e);
#pragma unroll
        for (int s = 0; s <= STAGES; ++s) {
            const uint32_t a = __shfl_sync(0xffffffffu, o0, s), b = __shfl_sync(0xffffffffu, o1, s);
            const uint32_t u = static_pos(s);
            if (s < STAGES) {
                item[s] = u;
                if (u < end && lane == 0 && u != p.withhold) {
                    const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
                    mbar_expect_tx(bar, (b - a) * 16u);
                    bulk_g2s(smem_u32(my_ring + (size_t)s * p.slot_bytes), p.blob + (size_t)a * 16u, (b - a) * 16u, bar, w_policy);
                }
            } else {
                ahead = u; po0 = a; po1 = b;
            }
        }
    }
    if (timing) dbg[1] = clock64() - t_start;
    if (threadIdx.x == 0) { claim[0] = beg + (uint32_t)n_static * (uint32_t)n_warps * R; claim[1] = 0; }
    if (AM && threadIdx.x < 64) amax_s[threadIdx.x] = 0;
    // refill slot s with the position fetched ahead
    auto refill = [&](int s) {
        if (lane == 0 && ahead < end && ahead != p.withhold) {
            const uint32_t bytes = (po1 - po0) * 16u;
            const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
            // the warp's earlier generic-proxy reads of this slot are ordered before the refill
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(bar, bytes);
            bulk_g2s(smem_u32(my_ring + (size_t)s * p.slot_bytes), p.blob + (size_t)po0 * 16u, bytes, bar, w_policy);
        }
        return ahead;
    };
    // take the next position and start fetching its offsets (called at the end of a tile's
    // bookkeeping: a fence issued after these loads would have to wait for them)
    auto fetch_ahead = [&]() {
        ahead = next_pos();
        if (lane == 0 && ahead < end) {
            const uint32_t i = ahead - beg;
            if (i < (uint32_t)kOffTable) {
                po0 = off_s[2 * i]; po1 = off_s[2 * i + 1];
            } else {
                const uint32_t t = tile_index(ahead);
                po0 = __ldg(p.item_off + t); po1 = __ldg(p.item_off + t + 1);
            }
        }
    };

    // Everything above (schedule, offsets, selector table, the first weight-tile copies) depends on
    // nothing an earlier kernel of the stream produces. X may be the output of the kernel before,
    // and Y / the workspace may still be in use by it: wait for the stream's earlier work here.
    int kr_first, kr_last, d0_, d1_;
    tile_of(beg, kr_first, d0_, d1_);
    tile_of(end - 1, kr_last, d0_, d1_);
    // Still independent of the stream's earlier work: the weight scales of the rows of this warp's
    // first strip (any warp may be the one that stores it; their row numbers were requested together
    // with the first offsets), the cleared sums and the table copies.
    ScalePre<NT> spre;
    if (kPreScales && pre_rb >= 0) {
        if (pre_mlo >= 0) spre.sw_lo = __ldg(p.w_scale + pre_mlo);
        if (pre_mhi >= 0) spre.sw_hi = __ldg(p.w_scale + pre_mhi);
        spre.rb = pre_rb;
    }
    auto clear_sums = [&]() {
        for (int i = threadIdx.x; i < p.G * NT * 8; i += blockDim.x) sx16[i] = 0;
        if (LA) {
            for (int i = threadIdx.x; i < p.s_local * NT * 128; i += blockDim.x) acc_l[i] = 0;
            for (int i = threadIdx.x; i < p.s_local; i += blockDim.x) cnt_l[i] = 0;
        }
        __syncthreads();
    };
    clear_sums();
    // copies of the selector table: entry e, copy r at word e * lut_rep + r (conflict-free writes)
    for (int i = threadIdx.x, sh = 31 - __clz(p.lut_rep); i < 256 * p.lut_rep; i += blockDim.x) lut[i] = lut1[i >> sh];

    asm volatile("griddepcontrol.wait;" ::: "memory");
    const unsigned long long g_wait = timing ? global_timer_ns() : 0;
    unsigned long long g_x = 0;
    // The activations of the CTA's first K range: fetch them into registers now, ahead of the
    // staging pass; and the activation scales of this lane's tokens.
    if (kPreScales && ScalePre<NT>::kSx && p.fp16_out) {
#pragma unroll
        for (int nt = 0; nt < (ScalePre<NT>::kSx ? NT : 1); ++nt)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int n = nt * 8 + (lane & 3) * 2 + j;
                spre.sx[nt][j] = n < p.N ? __ldg(p.x_scale + n) : (unsigned short)0;
            }
        spre.have_sx = true;
    }
    const int g_first = (kr_first == n_kr - 1) ? g_last : p.G;   // segments in that range
    constexpr int kXPre = NT <= 4 ? 8 : 0;   // 16-byte units of X a thread prefetches
    const int x_sh = 31 - __clz(p.K_L / 32);   // log2(units per (segment, token)) when a power of two
    const bool x_early = kXPre > 0 && p.x_fast == 2 && (1 << x_sh) == p.K_L / 32;
    uint4 xpre[kXPre > 0 ? kXPre : 1];
    const int x_upr = p.K_L / 32, x_total = NT * 8 * g_first * x_upr;
    if (x_early) {
        const int64_t ldx = ((int64_t)p.K + 1) / 2;
#pragma unroll
        for (int b = 0; b < kXPre; ++b) {
            const int u = threadIdx.x + b * blockDim.x;
            xpre[b] = make_uint4(0, 0, 0, 0);
            if (u < x_total) {
                const int pi = u >> x_sh, q = u & (x_upr - 1);
                const int sgl = pi / (NT * 8), n = pi & (NT * 8 - 1);
                const int64_t k = (int64_t)(kr_first * p.G + sgl) * p.K_L + 32 * q;
                if (n < p.N && k < p.K)
                    xpre[b] = __ldg(reinterpret_cast<const uint4*>(p.X + (int64_t)n * ldx + k / 2));
            }
        }
    }
    uint32_t phase = 0;   // bit s = parity to wait for on stage s
    bool dead = false;    // a bounded wait ran out: stop working, keep the barriers balanced
    int pend_rb = -1;     // direct mode: strip whose contribution is issued but not yet signalled
    uint32_t pend_n = 0;  //              and the number of tiles in it
    const int t2 = (lane & 3) * 2;
    const uint32_t lut_a = smem_u32(lut) + 4u * (uint32_t)(lane & (p.lut_rep - 1));

    const StoreCtx sctx{p.Y, p.w_scale, p.x_scale, p.acc, p.cnt, p.M, p.N, p.fp16_out,
                        AM ? amax_s : nullptr, p.amax_m0, p.amax_m1};
    auto store_strip = [&](int rb, int (&v)[NT][4], int m_lo, int m_hi) {
        if (m_lo == kNoRow) {   // not prefetched by the caller
            m_lo = __ldg(p.row_order + rb * 16 + (lane >> 2));
            m_hi = __ldg(p.row_order + rb * 16 + (lane >> 2) + 8);
        }
        store_rows<NT, AM>(sctx, v, lane, m_lo, m_hi, kPreScales ? &spre : nullptr, rb);
    };
    // add v to the global workspace of strip rb
    auto red_global = [&](int rb, int (&v)[NT][4]) {
        int32_t* accp = p.acc + (size_t)rb * (NT * 128) + lane;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) atomicAdd(accp + nt * 128 + j * 32, v[nt][j]);
    };
    // announce n_tiles finished contributions to strip rb; the arrival that completes it finalizes
    auto signal_strip = [&](int rb, uint32_t n_tiles, int m_lo, int m_hi) {
        // One acquire-release add instead of fence + add + fence: the warp barrier orders every
        // lane's adds to the workspace before lane 0's release; the arrival that completes the strip
        // acquires every earlier contributor's adds, and the second warp barrier hands that to the
        // other lanes. (Measured against the three-step form: N = 32 on 28672 x 8192 52.8 -> 48.8 us,
        // N = 8 on 8192 x 28672 28.7 -> 27.6 us.)
        __syncwarp();
        uint32_t old = 0;
        if (lane == 0)
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p.cnt + rb), "r"(n_tiles) : "memory");
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old + n_tiles == (uint32_t)p.n_segs) {
            __syncwarp();
            if (m_lo == kNoRow) {
                m_lo = __ldg(p.row_order + rb * 16 + (lane >> 2));
                m_hi = __ldg(p.row_order + rb * 16 + (lane >> 2) + 8);
            }
            finalize_strip<NT, AM>(sctx, rb, lane, m_lo, m_hi);
        }
    };

    int cur = 0;
    int rb = 0, sgl = 0, m_lo = kNoRow, m_hi = kNoRow;   // strip / segment / row ids of the tile in hand
    uint32_t last_u = 0xFFFFFFF0u;
    int y[NT][4];          // partial Y of the run in flight (fragment order)
    uint32_t y_n = 0;      // tiles summed in y
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) y[nt][0] = y[nt][1] = y[nt][2] = y[nt][3] = 0;

    // Stage the activations of K range kr: clear the sums, expand X, synchronise.
    auto stage_range = [&](int kr, int g_kr, bool first) {
        const bool use_prefetched = first && x_early;
        if (!first) clear_sums();
        if (use_prefetched) {
            // expand the prefetched units; anything beyond them goes through the general path
#pragma unroll
            for (int b = 0; b < kXPre; ++b) {
                const int u = threadIdx.x + b * blockDim.x;
                if (u < x_total) {
                    const int pi = u >> x_sh, q = u & (x_upr - 1);
                    const int sgl = pi / (NT * 8), n = pi & (NT * 8 - 1);
                    int32_t sacc = 0;
                    uint4 vlo, vhi;
                    uint2 t;
                    if (XP) {
                        vlo.x = pack8(xpre[b].x, sacc); vlo.y = pack8(xpre[b].y, sacc);
                        vlo.z = pack8(xpre[b].z, sacc); vlo.w = pack8(xpre[b].w, sacc);
                        *reinterpret_cast<uint4*>(x8 + n * xstride + (sgl * p.K_L + 32 * q) / 2) = vlo;
                    } else {
                        t = expand8(xpre[b].x, sacc); vlo.x = t.x; vlo.y = t.y;
                        t = expand8(xpre[b].y, sacc); vlo.z = t.x; vlo.w = t.y;
                        t = expand8(xpre[b].z, sacc); vhi.x = t.x; vhi.y = t.y;
                        t = expand8(xpre[b].w, sacc); vhi.z = t.x; vhi.w = t.y;
                        uint4* dst = reinterpret_cast<uint4*>(x8 + n * xstride + sgl * p.K_L + 32 * q);
                        dst[0] = vlo; dst[1] = vhi;
                    }
                    if (x_upr == 32) {   // one warp holds exactly one (segment, token) pair
                        sacc = __reduce_add_sync(0xffffffffu, sacc);
                        if (lane == 0) sx16[pi] = sacc;
                    } else if (sacc) {
                        atomicAdd(sx16 + pi, sacc);
                    }
                }
            }
            stage_x<NT, XP>(p, kr * p.G, g_kr, x8, xstride, sx16, kXPre * (int)blockDim.x);
        } else {
            stage_x<NT, XP>(p, kr * p.G, g_kr, x8, xstride, sx16, 0);
        }
        __syncthreads();
    };
    if (timing) dbg[2] = clock64() - t_start;
    // The first range is staged here, outside the loop, so that the prefetched X registers are
    // dead before the decode loop starts.
    stage_range(kr_first, g_first, true);
    if (timing) { dbg[3] = clock64() - t_start; g_x = global_timer_ns(); }

    for (int kr = kr_first; kr <= kr_last; ++kr) {
        const int g_kr = (kr == n_kr - 1) ? g_last : p.G;
        const unsigned long long mg = (kr == n_kr - 1) ? p.mg_glast : p.mg_g;
        const uint32_t base = (uint32_t)kr * kr_stride;
        const uint32_t lo = max(beg, base), hi = min(end, base + (uint32_t)p.n_strips * (uint32_t)g_kr);
        const uint32_t qlo = lo - base, qhi = hi - base;
        const int rb_first = (int)fdiv(qlo, mg);
        if (kr != kr_first) {
            __syncthreads();  // everyone is done with the previous range's X and sums
            stage_range(kr, g_kr, false);
        }
        if (timing && t_first == 0) t_first = clock64();

        while (!dead) {
            uint32_t u = 0;
#pragma unroll
            for (int s = 0; s < STAGES; ++s)
                if (s == cur) u = item[s];
            if (u >= hi) break;
            const long long t0 = timing ? clock64() : 0;
            const uint32_t bar = smem_u32(&bars[warp * STAGES + cur]);
            if (!mbar_wait_bounded(bar, (phase >> cur) & 1u, p.wait_ns_hi)) {
                if (lane == 0) atomicExch(p.err, kErrTimeout);
                dead = true;
                break;
            }
            phase ^= 1u << cur;
            const long long t1 = timing ? clock64() : 0;

            const uint32_t q = u - base;
            if (u == last_u + 1u && sgl + 1 < g_kr) {
                ++sgl;                         // next segment of the same strip
            } else {
                rb = (int)fdiv(q, mg);
                sgl = (int)(q - (uint32_t)rb * (uint32_t)g_kr);
                // original rows of this strip's fragment rows g and g + 8: needed only when the
                // strip is stored, fetched now so that the loads complete behind the decode
                m_lo = __ldg(p.row_order + rb * 16 + (lane >> 2));
                m_hi = __ldg(p.row_order + rb * 16 + (lane >> 2) + 8);
            }
            last_u = u;
            int c[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0;
            const uint32_t slot_a = smem_u32(my_ring + (size_t)cur * p.slot_bytes);
            const uint32_t xb_a = XP ? smem_u32(x8) + (lane >> 2) * xstride + 4 * (lane & 3) + sgl * (p.K_L / 2)
                                     : smem_u32(x8) + (lane >> 2) * xstride + 8 * (lane & 3) + sgl * p.K_L;
            if (DP) {
                const uint32_t xb0 = smem_u32(x8) + 8 * (lane & 3) + sgl * p.K_L;   // token 0, this lane's columns
                process_tile<NT, XP, CA, W2, true>(slot_a, lut_a, 4u * (uint32_t)p.lut_rep, xb0, xstride, p.mask_rows, lane, c, 0u);
                // the four lanes of a row group hold parts of the same two sums; the first keeps them in the
                // accumulator slots of token 0, the slots of tokens 1..7 stay zero
                int r = c[0][0], e = c[0][2];
                r += __shfl_xor_sync(0xffffffffu, r, 1); r += __shfl_xor_sync(0xffffffffu, r, 2);
                e += __shfl_xor_sync(0xffffffffu, e, 1); e += __shfl_xor_sync(0xffffffffu, e, 2);
                const bool first = (lane & 3) == 0;
                c[0][0] = first ? r : 0; c[0][2] = first ? e : 0;
            } else {
                process_tile<NT, XP, CA, W2>(slot_a, lut_a, 4u * (uint32_t)p.lut_rep, xb_a, xstride, p.mask_rows, lane, c,
                                             (uint32_t)p.fold_kb * (XP ? 16u : 32u));
            }
            __syncwarp();
            const long long t2c = timing ? clock64() : 0;

            // refill this slot right away, so that the copy overlaps the bookkeeping
            {
                const uint32_t issued = refill(cur);
#pragma unroll
                for (int s = 0; s < STAGES; ++s)
                    if (s == cur) item[s] = issued;
            }
            cur = (cur + 1 == STAGES) ? 0 : cur + 1;

            // ---- fragment sums -> partial Y of this tile, added to the run's sums ----
            const int32_t* sxp = sx16 + sgl * (NT * 8);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int n0 = nt * 8 + t2;
                const int s0 = sxp[n0] >> 4, s1 = sxp[n0 + 1] >> 4;
                if (W2) {
                    y[nt][0] += (c[nt][2] >> 4) - 2 * s0;                  // strip row g
                    y[nt][1] += (c[nt][3] >> 4) - 2 * s1;
                    y[nt][2] += ((c[nt][0] - c[nt][2]) >> 6) - 2 * s0;     // strip row g + 8
                    y[nt][3] += ((c[nt][1] - c[nt][3]) >> 6) - 2 * s1;
                } else {
                    y[nt][0] += (c[nt][2] >> 4) - 8 * s0;                 // strip row g
                    y[nt][1] += (c[nt][3] >> 4) - 8 * s1;
                    y[nt][2] += (c[nt][0] - c[nt][2]) >> 8;               // strip row g + 8
                    y[nt][3] += (c[nt][1] - c[nt][3]) >> 8;
                }
            }
            ++y_n;
            // the run goes on if this warp's next tile is the next segment of the same strip
            uint32_t u_next = 0;
#pragma unroll
            for (int s = 0; s < STAGES; ++s)
                if (s == cur) u_next = item[s];
            const bool more = (u_next == u + 1u) && (u_next < hi) && (sgl + 1 < g_kr);
            if (!more) {
                // what happens to the run's sums: 0 = nothing more, 1 = store (the strip is complete
                // here), 2 = add to the global workspace and announce `tell` tiles
                int action = 0;
                uint32_t tell = 0;
                if (LA) {
                    // tiles of this strip inside the CTA's part of the K range
                    const uint32_t expected = min(qhi, (uint32_t)(rb + 1) * (uint32_t)g_kr) - max(qlo, (uint32_t)rb * (uint32_t)g_kr);
                    bool flush = (y_n == expected);   // the whole of it was summed in registers
                    if (!flush) {
                        int32_t* al = acc_l + (rb - rb_first) * (NT * 128) + lane;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                            for (int j = 0; j < 4; ++j) atomicAdd(al + nt * 128 + j * 32, y[nt][j]);
                        // (one acquire-release add on the strip's counter instead of fence, add, fence:
                        // as for the global workspace below, with the warp barriers on both sides)
                        __syncwarp();
                        uint32_t old = 0;
                        if (lane == 0)
                            asm volatile("atom.acq_rel.cta.shared.add.u32 %0, [%1], %2;"
                                         : "=r"(old) : "r"(smem_u32(cnt_l + (rb - rb_first))), "r"(y_n) : "memory");
                        old = __shfl_sync(0xffffffffu, old, 0);
                        if (old + y_n == expected) {   // the CTA's last tiles of this strip: flush it
                            __syncwarp();
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                                for (int j = 0; j < 4; ++j) y[nt][j] = *(volatile int32_t*)(al + nt * 128 + j * 32);
                            flush = true;
                        }
                    }
                    if (flush) { action = (expected == (uint32_t)p.n_segs) ? 1 : 2; tell = expected; }
                } else if (p.n_segs == 1) {
                    action = 1;
                } else {
                    // The previous run's red.adds were issued a while ago: its fence is cheap now.
                    if (pend_rb >= 0) signal_strip(pend_rb, pend_n, kNoRow, kNoRow);
                    red_global(rb, y);
                    pend_rb = rb; pend_n = y_n;
                }
                if (action == 1) {
                    store_strip(rb, y, m_lo, m_hi);
                } else if (action == 2) {
                    red_global(rb, y);
                    signal_strip(rb, tell, m_lo, m_hi);
                }
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) y[nt][0] = y[nt][1] = y[nt][2] = y[nt][3] = 0;
                y_n = 0;
            }
            fetch_ahead();
            if (timing) {
                const long long t3 = clock64();
                t_wait += t1 - t0; t_decode += t2c - t1; t_epi += t3 - t2c;
            }
        }
    }
    if (pend_rb >= 0) signal_strip(pend_rb, pend_n, kNoRow, kNoRow);

    // Drain (only after a bounded wait ran out; in a normal run every issued tile was consumed):
    // copies this warp issued must land before the CTA exits.
    if (dead) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            if (item[s] < end && item[s] != p.withhold) {
                const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
                if (!mbar_wait_bounded(bar, (phase >> s) & 1u, p.wait_ns_hi) && lane == 0) atomicExch(p.err, kErrTimeout);
            }
        }
    }
    // Chained call: the last warp of the CTA to finish publishes the CTA's per-token absmax.
    if (AM) {
        __syncwarp();
        uint32_t old = 0;
        if (lane == 0)
            asm volatile("atom.acq_rel.cta.shared.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(smem_u32(claim + 1)) : "memory");
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old == (uint32_t)n_warps - 1u) {
            for (int n = lane; n < 64; n += 32)
                p.y_amax[64 + 64 * blockIdx.x + n] = n < NT * 8 ? *(volatile uint32_t*)(amax_s + n) : 0u;
            if (blockIdx.x == 0 && lane == 0) p.y_amax[0] = gridDim.x;
        }
    }
    if (timing && lane == 0) {
        // one record per warp, plain stores (contended atomics here would hold up the warps still
        // decoding: global and shared-memory instructions share the SM's memory pipeline)
        unsigned long long* R = p.timers + (size_t)kWarpRec * ((size_t)blockIdx.x * kMaxWarpsPerCta + (size_t)warp);
        R[1] = (unsigned long long)t_wait; R[2] = (unsigned long long)t_decode; R[3] = (unsigned long long)t_epi;
        R[4] = (unsigned long long)(clock64() - t_start); R[5] = (unsigned long long)(t_first - t_start);
        R[6] = g_start; R[7] = g_x; R[8] = (unsigned long long)global_timer_ns();
        R[9] = (unsigned long long)dbg[0]; R[10] = (unsigned long long)dbg[1]; R[11] = (unsigned long long)dbg[2];
        R[12] = (unsigned long long)dbg[3]; R[13] = g_wait;
        R[0] = 1ull;
    }
}

}  // namespace us
