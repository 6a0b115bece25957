// C ABI of the library (declared in include/unionsparse.h): handle management, upload, launch.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "us_host.h"
#include "us_spmm_kernel.cuh"
#include "us_quant_kernels.cuh"

struct us_handle {
    us::HostMatrix host;
    bool on_device = false;
    int device = -1;
    int sm_count = 0;
    int max_N = 0;
    int max_smem = 0;
    int co_warps = 10;   // warps of an N <= 8 CTA when two CTAs share an SM's registers
    int co_warps2 = 8;   // the same for the N = 9..16 kernel with packed activations
    int co_warps_fold = 8;   // the same for the folded-tile (two column areas) N <= 8 kernel
    uint8_t* d_blob = nullptr;
    uint32_t* d_item_off = nullptr;
    std::vector<uint32_t> cta_begin[4];  // schedule per N class (NT = 1, 2, 4, 8)
    int G[4] = {1, 1, 1, 1};          // segments per K range, per class
    int s_local[4] = {0, 0, 0, 0};    // strips held in shared memory (0 = direct mode), per class
    bool xp[4] = {false, false, false, false};   // X staged packed (half the shared memory), per class
    int32_t* d_row_order = nullptr;
    uint16_t* d_w_scale = nullptr;
    int32_t* d_acc = nullptr;
    uint32_t* d_cnt = nullptr;
    uint32_t* d_err = nullptr;
    uint8_t* d_xq = nullptr;          // chained calls: packed INT4 codes of the activations, then their scales
    size_t xq_bytes = 0;              // bytes of the codes (the fp16 scales follow, 256-byte aligned)
    unsigned long long* d_timers = nullptr;
    bool timers_on = false;
    size_t acc_bytes = 0, cnt_bytes = 0;
    uint32_t withhold = 0xFFFFFFFFu;   // test hook (us_debug_withhold_copy)
    uint32_t wait_ns_hi = 2000000u;    // bounded waits: ~2 s
    cudaError_t sticky = cudaSuccess;
};

namespace {


int nt_for(int N) { return N <= 8 ? 1 : N <= 16 ? 2 : N <= 32 ? 4 : 8; }
int class_of(int nt) { return nt == 1 ? 0 : nt == 2 ? 1 : nt == 4 ? 2 : 3; }

// Experiment knobs, overridable from the environment (read once per process). Everything else the
// plan decides from the shape.
int env_int(const char* name, int fallback)
{
    const char* v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : fallback;
}
int pdl_knob() { static int v = env_int("US_PDL", 1); return v; }          // programmatic dependent launch
int stages_knob() { static int v = env_int("US_STAGES", 0); return v; }    // ring slots per warp, 0 = automatic
// (up to 20 for the N <= 8 kernels; the other kernels are compiled for 16)
int max_warps() { static int v = std::min(20, std::max(2, env_int("US_MAX_WARPS", 16))); return v; }
int coresident_knob() { static int v = env_int("US_CORESIDENT", 1); return v; }  // small problems: half an SM per CTA
constexpr int kLocalAccBudget = 32 * 1024;   // local strip sums a K-range width is chosen with
constexpr int kLocalAccCap = 48 * 1024;      // ... and what is taken if nothing fits that
constexpr int kMinWarps = 12;                // warps the automatic K-range choice keeps room for
constexpr int kCoresidentTiles = 16;         // most tiles per CTA for the half-SM plan
constexpr int kHalfSmBytes = 228 * 1024 / 2 - 1024 - 512;   // shared memory of a half-SM CTA: 228 KB per SM, 1 KB reserved per CTA

struct LaunchGeom {
    int nt, cls, warps, stages, smem, lut_rep;
    uint32_t slot_bytes;
    bool xp;
};

// Segments per K range for an N class. The int8 activations of one K range live in shared memory
// next to the warps' tile slots, so fewer, longer ranges (fewer partial-sum flushes) cost warps.
// Returns the range length of the split into the fewest equal ranges, not fewer than min_ranges,
// that still leaves room for min_warps one-slot warps (measured: 15 warps and one range beat
// 16 warps and two ranges by 25 % on a 13824 x 5120 matrix at N = 16).
// Shared memory of one K range's activations: int8 (one byte per token and k, 32 bytes of pad per
// token row) or packed (half of that).
// Ring slot: the largest tile plus the two payload rows the decode's window loads may read past a
// stream's end (rows are 128 bytes per column area).
uint32_t slot_bytes_for(const us::HostMatrix& hm)
{
    const uint32_t streams = hm.w2 ? 1u : (uint32_t)hm.fmt.C_A;
    return (hm.max_item_bytes + 256u * streams + 127u) & ~127u;
}

int64_t x_bytes(int nt, int64_t G, int K_L, bool xp)
{
    return xp ? (int64_t)nt * 8 * (G * K_L / 2 + 16) : (int64_t)nt * 8 * (G * K_L + 32);
}

int segs_per_range(const us::HostMatrix& hm, int nt, int limit, int64_t min_ranges, bool xp)
{
    const int64_t n_segs = hm.n_segs;
    const int slot = (int)slot_bytes_for(hm);
    const int acc = nt * 512 * 2 <= kLocalAccBudget ? kLocalAccBudget : 0;
    const int other = 256 * 8 * 4 + (int)us::kLutScratchBytes + acc + 2 * us::kOffTable * 4 + 1280;
    for (int64_t r = std::max<int64_t>(1, min_ranges); r <= n_segs; ++r) {
        // A single range is worth more (no partial sums leave the CTA when the cuts fall on strip
        // boundaries): it may cost two more warps. Measured on 4096 x 11008, N = 8: one range with
        // 15 warps 9.8 us, two ranges with 16 warps 14.7 us.
        const int want = std::min(max_warps(), r == 1 ? std::min(10, kMinWarps) : kMinWarps);
        const int64_t G = (n_segs + r - 1) / r;
        const int64_t xb = x_bytes(nt, G, hm.fmt.K_L, xp) + G * nt * 32;
        if ((limit - other - xb) / slot >= want) return (int)G;
    }
    return 1;
}

// Shared-memory layout of us_spmm_kernel: selector table, int8 X of one K range, per-(segment,
// token) sums, mbarriers, claim counter, local strip accumulators + counters, per-warp rings.
bool plan_launch(const us_handle* h, int N, LaunchGeom* g)
{
    g->nt = nt_for(N);
    g->cls = class_of(g->nt);
    const int G = h->G[g->cls], s_local = h->s_local[g->cls];
    g->xp = h->xp[g->cls];
    g->slot_bytes = slot_bytes_for(h->host);
    // selector table copies: 32 (conflict-free lookups) when that costs no warp, else 8
    int lut_rep = 32;
    auto fixed_for = [&](int rep) {
        return 256 * rep * 4 + (int)us::kLutScratchBytes + (int)x_bytes(g->nt, G, h->host.fmt.K_L, g->xp) + G * g->nt * 8 * 4 +
                           us::kClaimWords * 4 + s_local * (g->nt * 128 + 1) * 4 + 2 * us::kOffTable * 4 + 128;
    };
    int fixed_base = fixed_for(lut_rep);
    const int limit = h->max_smem > 0 ? h->max_smem : 227 * 1024;
    // Ring depth: two slots per warp when that still gives (nearly) all the warps; else one slot per
    // warp and more warps -- measured on the 70B-shaped FFN: 16 warps x 1 slot beat 9 warps x 2.
    auto warps_for = [&](int stages) {
        const int fixed = fixed_base + 32 * stages * 8;
        return std::min((limit - fixed) / (int)(stages * g->slot_bytes),
                        (g->nt == 1 && h->host.fmt.C_A == 1) ? max_warps() : std::min(16, max_warps()));
    };
    {
        const int w32 = std::max(warps_for(1), warps_for(2));
        fixed_base = fixed_for(8);
        const int w8 = std::max(warps_for(1), warps_for(2));
        // 32 copies only for long-running CTAs (measured: 1 % faster on the 70B-shaped FFN, but the
        // 4096 x 4096 case -- about one tile per warp -- loses 5 % to the bigger table)
        const int64_t n_cta = h->sm_count > 0 ? h->sm_count : 148;
        const bool long_run = (h->host.n_items + n_cta - 1) / n_cta >= 4 * (int64_t)w8;
        if (w32 >= w8 && long_run) { lut_rep = 32; fixed_base = fixed_for(32); } else { lut_rep = 8; }
    }
    int stages = stages_knob() > 0 ? stages_knob() : (warps_for(1) >= warps_for(2) + 3 ? 1 : 2);
    int warps = warps_for(stages);
    if (warps < 2) return false;
    // Small problems at N <= 8 (a CTA sees about a tile per warp): take at most half an SM -- shared
    // memory and registers -- with one slot per warp, so that the next launch's CTA moves in beside
    // this one and runs its latency-bound prologue (parameters, offsets, first tile copies, table)
    // under this one's work; with one CTA per SM, programmatic dependent launch alone hides only the
    // launch latency, because all CTAs of a launch end at about the same time.
    // Measured on 4096 x 4096, N = 8: 6.6 -> 5.7 us; not worth it from ~20 tiles per CTA on.
    const int64_t n_cta = h->sm_count > 0 ? h->sm_count : 148;
    const int64_t per_cta = (h->host.n_items + n_cta - 1) / n_cta;
    int fixed = fixed_base + 32 * stages * 8;
    // (N = 9..16 too, where the plan stages X packed and in local mode: that kernel is as lean.)
    // (Tried at N = 32 as well: 8 warps per CTA, slower.)
    const bool co_class = g->nt == 1 || (g->nt == 2 && g->xp && s_local > 0);
    if (coresident_knob() && co_class && per_cta <= kCoresidentTiles && stages_knob() == 0) {
        const int half = kHalfSmBytes;
        const int fixed8 = fixed_for(8) + 32 * 8;
        const bool fold = h->host.fmt.C_A == 2;
        int w = std::min(g->nt == 1 ? (fold ? h->co_warps_fold : h->co_warps) : h->co_warps2,
                         (g->nt == 1 && !fold) ? max_warps() : std::min(16, max_warps()));
        while (w >= 8 && fixed8 + w * (int)g->slot_bytes > half) --w;
        // (only if nearly every tile of the CTA finds a warp at once: 5120 x 5120 at 70 % sparsity, N = 16, has 11
        // tiles per CTA and room for 8 half-SM warps: 9.9 us against 8.9 with 16 warps on the whole SM)
        if (w >= 8 && w >= std::min<int64_t>(per_cta, 10)) { stages = 1; lut_rep = 8; warps = w; fixed = fixed8; }
    }
    g->stages = stages;
    g->lut_rep = lut_rep;
    g->warps = warps;
    g->smem = fixed + warps * stages * (int)g->slot_bytes;
    return true;
}

// Chooses, per N class, the K-range width, whether strips are summed in shared memory, and whether
// X is staged packed.
void plan_classes(us_handle* h, int n_cta, std::vector<uint32_t> (&sched)[4])
{
    const int limit = h->max_smem > 0 ? h->max_smem : 227 * 1024;
    for (int c = 0; c < 4; ++c) {
        const int nt = 1 << c;
        // Local mode needs the strip sums of a CTA's share of one K range in shared memory; a short
        // last range spreads a CTA over more strips, so shorter ranges are tried before giving up.
        // Returns the range length found (0 = none) and leaves the schedule in `out`.
        auto local_plan = [&](bool xp, std::vector<uint32_t>* out, int* s_local) -> int {
            // second pass: a little more than the budget the range length was chosen with is taken
            // if nothing fits the budget and at least 11 warps remain -- the alternative is the global
            // split-K path for every tile (N = 32: 5120 x 13824 30.2 -> 22.4 us, 4096 x 11008 18.7 ->
            // 16.2 us; N = 64 on 5120 x 5120 25.3 -> 19.5 us)
            for (int pass = 0; pass < 2; ++pass) {
                int G = 0, worst = 1;
                for (int64_t r = 1; r <= h->host.n_segs; ++r) {
                    const int Gr = segs_per_range(h->host, nt, limit, r, xp);
                    if (Gr == G) continue;
                    G = Gr;
                    if (G <= 1) break;
                    us::make_schedule(h->host, n_cta, G, out, &worst);
                    const int need = worst * nt * 512;
                    if (pass == 0 && need <= kLocalAccBudget) { *s_local = worst; return G; }
                    if (pass == 1 && need <= kLocalAccCap) {
                        const int slot = (int)slot_bytes_for(h->host);
                        const int64_t fixed = 256 * 8 * 4 + (int64_t)us::kLutScratchBytes + need + 2 * us::kOffTable * 4 + 1280 +
                                              x_bytes(nt, G, h->host.fmt.K_L, xp) + (int64_t)G * nt * 32;
                        if ((limit - fixed) / slot >= 11) { *s_local = worst; return G; }
                    }
                }
            }
            return 0;
        };
        h->G[c] = 1;
        h->s_local[c] = 0;
        h->xp[c] = false;
        int sl = 0;
        const int G = local_plan(false, &sched[c], &sl);
        if (G > 0) { h->G[c] = G; h->s_local[c] = sl; }
        // Packed X (N <= 32: the kernel exists for those classes) halves the shared memory of a K
        // range at the price of three more integer instructions per n-tile and k-block. Worth it
        // when it turns several K ranges into one (then no partial sum leaves the CTA; N = 8 on
        // 5120 x 13824: 18.2 -> 15.1 us; where one range was enough already it costs 2-6 %).
        // Measured at N = 16: 28672 x 8192 38.4 -> 34.8 us and 4096 x 11008 17.9 -> 14.4 us (two
        // ranges become one); 5120 x 5120 12.0 -> 9.4 us (one range either way, but a CTA's share is
        // small and the staging pass and the freed shared memory count for more than the decode);
        // 13824 x 5120 15.7 -> 16.0 us (one range either way, long decode): not taken there.
        if (nt <= 4 && !h->host.w2) {   // (no packed-X kernel for INT2 weights)
            const int64_t n_segs = h->host.n_segs;
            const int64_t ranges = h->s_local[c] > 0 ? (n_segs + h->G[c] - 1) / h->G[c] : n_segs + 1;
            const bool small_share = nt >= 2 && (int64_t)h->host.blob.size() / std::max(1, n_cta) < 128 * 1024;
            // N <= 8: packed X when that is what lets the half-SM plan of plan_launch hold its eight warps
            // (4096 x 4096 at 30 % sparsity: tiles of 9.5 KB and 32 KB of int8 X do not fit half an SM, with
            // 16 KB of packed X they do: 5.6 -> 4.6 us; the same for the folded format at 50 %: 5.3 -> 4.35)
            bool for_half_sm = false;
            if (nt == 1 && ranges == 1 && coresident_knob()) {
                const int64_t per_cta = (h->host.n_items + n_cta - 1) / std::max(1, n_cta);
                const int64_t need = 8;
                auto fits = [&](bool xp, int s_loc) {
                    const int64_t fixed8 = 256 * 8 * 4 + (int64_t)us::kLutScratchBytes + x_bytes(nt, n_segs, h->host.fmt.K_L, xp) +
                                           n_segs * nt * 8 * 4 + us::kClaimWords * 4 + (int64_t)s_loc * (nt * 128 + 1) * 4 +
                                           2 * us::kOffTable * 4 + 128 + 32 * 8;
                    return fixed8 + need * (int64_t)slot_bytes_for(h->host) <= kHalfSmBytes;
                };
                // (only where every tile then finds its own warp: 5120 x 5120 at 70 % sparsity, 11 tiles per CTA,
                // runs 7.7 us in a 12-warp half-SM CTA against 6.3 us with 16 warps on the whole SM)
                for_half_sm = per_cta <= 8 && !fits(false, h->s_local[c]) && fits(true, h->s_local[c]);
            }
            if (ranges > 1 || small_share || for_half_sm) {
                std::vector<uint32_t> alt;
                int sl2 = 0;
                const int G2 = local_plan(true, &alt, &sl2);
                const int64_t ranges2 = G2 > 0 ? (n_segs + G2 - 1) / G2 : 0;
                // (N = 32, packed against plain: 11008 x 4096 21.4 -> 18.5 us, 13824 x 5120 24.9 -> 23.6 us,
                // 5120 x 5120 17.3 -> 18.2 us with one range; three ranges instead of eleven one-segment
                // ranges on 4096 x 11008 were slower, 19.3 -> 26.4 us: only a single range pays)
                if (G2 > 0 && ranges2 == 1) {
                    h->G[c] = G2; h->s_local[c] = sl2; h->xp[c] = true;
                    sched[c] = alt;
                }
            }
        }
        // direct mode: one segment per range, every tile goes to the global workspace (longer ranges
        // and runs were measured: no gain at N = 32, the bigger X costs more than the adds it saves)
        int worst = 1;
        if (h->s_local[c] == 0) us::make_schedule(h->host, n_cta, 1, &sched[c], &worst);
    }
}

template <int NT, int ST>
cudaError_t launch_st(const us::SpmmParams& p, bool xp, int grid, int block, int smem, cudaStream_t st)
{
    // Launched with programmatic stream serialization: the kernel may start while its predecessor
    // in the stream is still running; it waits (griddepcontrol.wait) before it touches anything
    // an earlier kernel could produce or still use.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_knob() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool la = p.s_local > 0, timed = p.timers != nullptr;
    if (p.w2)   // INT2 weights in folded tiles: plain kernels only (no packed X, timers or absmax)
        return la ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, true, false, false, false, 2, true>, p)
                  : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, false, false, false, false, 2, true>, p);
    if (p.fold_kb) {   // folded tiles (two column areas); stage timers for the N <= 8 kernels only
        if (NT == 1 && timed && !xp)
            return la ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<1, ST, true, true, false, false, 2>, p)
                      : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<1, ST, false, true, false, false, 2>, p);
        if (NT <= 4 && xp && la) {
            constexpr int NP = NT <= 4 ? NT : 4;
            return cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NP, ST, true, false, true, false, 2>, p);
        }
        return la ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, true, false, false, false, 2>, p)
                  : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, false, false, false, false, 2>, p);
    }
    if (p.y_amax) {   // chained call (never timed: enqueue_spmm leaves the timers off)
        if (NT <= 4 && xp && la) {
            constexpr int NP = NT <= 4 ? NT : 4;
            return cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NP, ST, true, false, true, true>, p);
        }
        return la ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, true, false, false, true>, p)
                  : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, false, false, false, true>, p);
    }
    if (NT <= 4 && xp && la) {   // packed X: planned for these classes and local mode only
        constexpr int NP = NT <= 4 ? NT : 4;
        return timed ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NP, ST, true, true, true>, p)
                     : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NP, ST, true, false, true>, p);
    }
    if (NT == 1 && p.N == 1 && !timed)   // a single token: dp4a beats the MMA (measured 2-3 %)
        return la ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<1, ST, true, false, false, false, 1, false, true>, p)
                  : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<1, ST, false, false, false, false, 1, false, true>, p);
    if (la && !timed) return cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, true, false>, p);
    if (!la && !timed) return cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, false, false>, p);
    if (la) return cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, true, true>, p);
    return cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NT, ST, false, true>, p);
}

template <int NT>
cudaError_t launch_nt(const us::SpmmParams& p, bool xp, int stages, int grid, int block, int smem, cudaStream_t st)
{
    return stages == 1 ? launch_st<NT, 1>(p, xp, grid, block, smem, st) : launch_st<NT, 2>(p, xp, grid, block, smem, st);
}

// Opt every kernel variant in to the device's full dynamic shared memory (once per handle, at
// encode time, so that us_spmm itself is nothing but a launch).
template <int NT, int ST>
cudaError_t enable_large_smem_st(int bytes)
{
    const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, true, false>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, false, false>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, true, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, true, false, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, false, false, false, true>, attr, bytes);
    constexpr int NP = NT <= 4 ? NT : 4;   // packed-X kernels exist for N <= 32
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NP, ST, true, false, true, true>, attr, bytes);
    if (NT == 1) {   // single-token kernels
        if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, ST, true, false, false, false, 1, false, true>, attr, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, ST, false, false, false, false, 1, false, true>, attr, bytes);
    }
    // folded tiles, INT4 and INT2
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, true, false, false, false, 2, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, false, false, false, false, 2, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, true, false, false, false, 2>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, ST, false, false, false, false, 2>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NP, ST, true, false, true, false, 2>, attr, bytes);
    if (NT == 1) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, ST, true, true, false, false, 2>, attr, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, ST, false, true, false, false, 2>, attr, bytes);
    }
    return e;
}
template <int NT>
cudaError_t enable_large_smem_nt(int bytes)
{
    cudaError_t e = enable_large_smem_st<NT, 1>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_st<NT, 2>(bytes);
    return e;
}
cudaError_t enable_large_smem(int bytes)
{
    cudaError_t e = enable_large_smem_nt<1>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_nt<2>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_nt<4>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_nt<8>(bytes);
    const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<2, 1, true, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<2, 2, true, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<2, 1, true, true, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<2, 2, true, true, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, 1, true, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, 2, true, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, 1, true, true, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<1, 2, true, true, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<4, 1, true, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<4, 2, true, false, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<4, 1, true, true, true>, attr, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<4, 2, true, true, true>, attr, bytes);
    return e;
}

void free_device(us_handle* h)
{
    cudaFree(h->d_blob); cudaFree(h->d_item_off);
    cudaFree(h->d_row_order); cudaFree(h->d_w_scale); cudaFree(h->d_acc);
    cudaFree(h->d_cnt); cudaFree(h->d_err); cudaFree(h->d_timers); cudaFree(h->d_xq);
}

template <class T>
cudaError_t upload(T** dst, const void* src, size_t bytes)
{
    cudaError_t e = cudaMalloc((void**)dst, std::max<size_t>(bytes, 16));
    if (e != cudaSuccess) return e;
    return bytes ? cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) : cudaSuccess;
}


// Argument checks shared by the two SpMM entry points.
us_status check_spmm_args(const us_handle* h, const void* X, int32_t N, const void* x_scale, const void* Y)
{
    if (!h || !X || !Y || N < 1 || N > h->max_N) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (x_scale && !h->d_w_scale) return US_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X) % 16) return US_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return US_ERR_CUDA;
    if (dev != h->device) return US_ERR_INVALID_ARG;   // the handle's arrays live on another GPU
    return US_OK;
}

// Fills the kernel parameters and launches: the one code path behind us_spmm and
// us_spmm_static_scratch (they differ only in where the split-K scratch lives).
// What a chained call adds to the plain one: the per-token absmax of a range of output rows, left
// for the quantiser of the next call.
struct ChainArgs {
    void* y_amax = nullptr;
    int64_t m0 = 0, m1 = 0;
};

us_status enqueue_spmm(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y, cudaStream_t st,
                       int32_t* acc, uint32_t* cnt, bool timers, const ChainArgs* chain = nullptr)
{
    LaunchGeom g;
    if (!plan_launch(h, N, &g)) return US_ERR_UNSUPPORTED;
    const us::HostMatrix& hm = h->host;
    us::SpmmParams p;
    p.blob = h->d_blob; p.item_off = h->d_item_off;
    std::memcpy(p.cta_begin, h->cta_begin[g.cls].data(), h->cta_begin[g.cls].size() * sizeof(uint32_t));
    p.G = h->G[g.cls]; p.s_local = h->s_local[g.cls]; p.lut_rep = g.lut_rep;
    {
        const int64_t n_kr = (hm.n_segs + p.G - 1) / p.G;
        const int64_t g_last = hm.n_segs - (n_kr - 1) * p.G;
        auto magic = [](uint64_t d) { return ((1ull << 40) / d) + 1ull; };
        p.mg_g = magic((uint64_t)p.G);
        p.mg_glast = magic((uint64_t)g_last);
        p.mg_krs = magic((uint64_t)hm.n_strips * (uint64_t)p.G);
        // Claim runs of up to a whole strip's segments of the range (the partial sums of a run stay
        // in registers; the kernel shortens the runs towards the end of a CTA's range), but never
        // so long that a CTA's warps run out of runs to share.
        const int64_t per_cta = std::max<int64_t>(1, hm.n_items / std::max(1, h->sm_count));
        const int balanced = (int)std::max<int64_t>(1, per_cta / (4 * (int64_t)g.warps));
        p.run_len = std::max(1, std::min(std::min(p.G, 2 * balanced), p.G));
        // Fewer tiles than warps: one tile per warp, all at once (1024 x 1024, N = 8: 4.1 -> 3.1 us); with more
        // tiles than warps, runs of two keep a run's sums in registers and win (4096 x 4096: 5.7 against 6.3 us).
        if ((hm.n_items + h->sm_count - 1) / std::max(1, h->sm_count) <= g.warps) p.run_len = 1;
    }
    p.row_order = h->d_row_order; p.w_scale = h->d_w_scale;
    p.X = static_cast<const uint8_t*>(X);
    p.x_scale = static_cast<const uint16_t*>(x_scale);
    p.Y = Y; p.acc = acc; p.cnt = cnt; p.err = h->d_err;
    // (no stage-timer builds of the absmax-tracking kernels, nor of the folded-tile kernels for N > 8 or with packed X:
    // a timer build launched on a plan laid out for another variant would index shared memory wrongly)
    p.timers = (timers && !(chain && chain->y_amax) && !(hm.fmt.C_A == 2 && (g.nt > 1 || g.xp)) && !hm.w2) ? h->d_timers : nullptr;
    p.M = (int32_t)hm.M; p.K = (int32_t)hm.K; p.N = N;
    p.n_strips = (int32_t)hm.n_strips; p.n_segs = (int32_t)hm.n_segs;
    p.mask_rows = hm.mask_rows; p.K_L = hm.fmt.K_L;
    p.fold_kb = hm.fmt.C_A == 2 ? hm.nkb / 2 : 0;
    p.w2 = hm.w2 ? 1 : 0;
    p.slot_bytes = g.slot_bytes;
    p.x_fast = (hm.K % 32 == 0) ? 2 : (hm.K % 8 == 0) ? 1 : 0;
    p.fp16_out = x_scale ? 1 : 0;
    p.y_amax = nullptr; p.amax_m0 = p.amax_m1 = 0;
    if (chain) {
        p.y_amax = static_cast<uint32_t*>(chain->y_amax);
        p.amax_m0 = (int32_t)chain->m0; p.amax_m1 = (int32_t)chain->m1;
    }
    p.wait_ns_hi = h->wait_ns_hi;
    p.withhold = h->withhold;

    cudaError_t e;
    switch (g.nt) {
        case 1: e = launch_nt<1>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
        case 2: e = launch_nt<2>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
        case 4: e = launch_nt<4>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
        default: e = launch_nt<8>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
    }
    if (e != cudaSuccess) { h->sticky = e; return US_ERR_CUDA; }
    return US_OK;
}

}  // namespace

extern "C" {

us_status us_encode(const int8_t* W, int64_t M, int64_t K, const uint16_t* w_scale,
                    const us_format* fmt, int32_t max_N, uint32_t flags, us_handle** out)
{
    if (out) *out = nullptr;
    if (!W || !out || M <= 0 || K <= 0 || max_N < 1 || max_N > 64) return US_ERR_INVALID_ARG;
    if (M > 0x7FFFFFF0ll || K > 0x7FFFFFF0ll) return US_ERR_INVALID_ARG;
    us_handle* h = new (std::nothrow) us_handle();
    if (!h) return US_ERR_ALLOC;
    h->max_N = max_N;
    const bool host_only = (flags & US_ENCODE_HOST_ONLY) != 0;
    cudaError_t e = cudaSuccess;
    if (!host_only) {
        e = cudaGetDevice(&h->device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device);
        if (e != cudaSuccess) { delete h; return US_ERR_CUDA; }
        if (h->sm_count > us::kMaxCtas) h->sm_count = us::kMaxCtas;
    }
    const int n_cta = h->sm_count > 0 ? h->sm_count : 148;   // host-only handles plan for a 148-SM part
    us_format f = fmt ? *fmt : us_format{16, us::default_K_L(M, K, n_cta), 2, 1};
    us_status s;
    try {
        s = us::encode_host(W, M, K, w_scale, f, flags, 0, &h->host);
    } catch (const std::bad_alloc&) {
        s = US_ERR_ALLOC;
    }
    if (s != US_OK) { delete h; return s; }
    const us::HostMatrix& hm = h->host;
    if (!hm.kernel_layout) {   // a format without a kernel: statistics and decoding only
        *out = h;
        return US_OK;
    }
    // the kernel's index arithmetic (exact division by multiplication) needs u * d < 2^40 for every
    // position u < n_items and divisor d <= n_items
    if (hm.n_items >= (1 << 20) || hm.n_segs >= (1 << 16)) {
        delete h;
        return US_ERR_UNSUPPORTED;
    }
    std::vector<uint32_t> sched[4];
    plan_classes(h, n_cta, sched);
    if (host_only) {
        *out = h;
        return US_OK;
    }

    e = enable_large_smem(h->max_smem);
    if (e == cudaSuccess) {
        // Two N <= 8 CTAs share the SM's 64 K registers (allocated 8 per thread at a time).
        int regs = 0;
        // (the stage-timer builds need more and simply do not share an SM)
        for (const void* fn : {(const void*)us::us_spmm_kernel<1, 1, true, false>, (const void*)us::us_spmm_kernel<1, 1, false, false>}) {
            cudaFuncAttributes fa;
            e = cudaFuncGetAttributes(&fa, fn);
            if (e != cudaSuccess) break;
            regs = std::max(regs, fa.numRegs);
        }
        if (e == cudaSuccess) h->co_warps = 32768 / (32 * ((regs + 7) / 8 * 8));
        cudaFuncAttributes fa2;
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa2, (const void*)us::us_spmm_kernel<2, 1, true, false, true>);
        if (e == cudaSuccess) h->co_warps2 = 32768 / (32 * ((fa2.numRegs + 7) / 8 * 8));
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa2, (const void*)us::us_spmm_kernel<1, 1, true, false, false, false, 2>);
        if (e == cudaSuccess) h->co_warps_fold = 32768 / (32 * ((fa2.numRegs + 7) / 8 * 8));
    }
    if (e != cudaSuccess) { delete h; return US_ERR_CUDA; }

    const int nt_max = nt_for(max_N);
    h->acc_bytes = (size_t)hm.n_strips * nt_max * 128 * sizeof(int32_t);
    h->cnt_bytes = (size_t)hm.n_strips * sizeof(uint32_t);
    e = upload(&h->d_blob, hm.blob.data(), hm.blob.size());
    if (e == cudaSuccess) e = upload(&h->d_item_off, hm.item_off.data(), hm.item_off.size() * 4);
    for (int c = 0; c < 4; ++c) h->cta_begin[c] = sched[c];
    if (e == cudaSuccess) e = upload(&h->d_row_order, hm.row_order.data(), hm.row_order.size() * 4);
    if (e == cudaSuccess && !hm.w_scale.empty()) e = upload(&h->d_w_scale, hm.w_scale.data(), hm.w_scale.size() * 2);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_acc, h->acc_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->d_acc, 0, h->acc_bytes);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_cnt, h->cnt_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->d_cnt, 0, h->cnt_bytes);
    if (e == cudaSuccess && !hm.w_scale.empty()) {   // chained calls need fp16 output, hence weight scales
        h->xq_bytes = (((size_t)max_N * (size_t)((hm.K + 1) / 2)) + 255) & ~(size_t)255;
        e = cudaMalloc((void**)&h->d_xq, h->xq_bytes + 256);
    }
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_err, 16);
    if (e == cudaSuccess) e = cudaMemset(h->d_err, 0, 16);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        free_device(h);
        delete h;
        cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? US_ERR_ALLOC : US_ERR_CUDA;
    }
    h->on_device = true;
    LaunchGeom g;
    if (!plan_launch(h, max_N, &g)) {  // a tile does not fit the shared-memory ring
        free_device(h);
        delete h;
        return US_ERR_UNSUPPORTED;
    }
    *out = h;
    return US_OK;
}

us_status us_get_stats(const us_handle* h, us_stats* out)
{
    if (!h || !out) return US_ERR_INVALID_ARG;
    us::fill_stats(h->host, out);
    return US_OK;
}

us_status us_decode(const us_handle* h, int8_t* W_out)
{
    if (!h || !W_out) return US_ERR_INVALID_ARG;
    us::decode_host(h->host, W_out);
    return US_OK;
}

us_status us_get_row_order(const us_handle* h, int32_t* perm_out)
{
    if (!h || !perm_out) return US_ERR_INVALID_ARG;
    if (!h->host.kernel_layout) {   // the paper's layout keeps the rows where they are
        for (int64_t r = 0; r < h->host.Mp; ++r) perm_out[r] = r < h->host.M ? (int32_t)r : -1;
        return US_OK;
    }
    std::memcpy(perm_out, h->host.row_order.data(), h->host.row_order.size() * sizeof(int32_t));
    return US_OK;
}

us_status us_launch_info(const us_handle* h, int32_t N, int32_t* grid, int32_t* block,
                         int32_t* smem_bytes)
{
    if (!h || N < 1 || N > h->max_N) return US_ERR_INVALID_ARG;
    if (!h->host.kernel_layout) return US_ERR_UNSUPPORTED;
    LaunchGeom g;
    if (!plan_launch(h, N, &g)) return US_ERR_UNSUPPORTED;
    if (grid) *grid = h->sm_count > 0 ? h->sm_count : 148;
    if (block) *block = g.warps * 32;
    if (smem_bytes) *smem_bytes = g.smem;
    return US_OK;
}

us_status us_spmm(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y, void* stream)
{
    const us_status s = check_spmm_args(h, X, N, x_scale, Y);
    if (s != US_OK) return s;
    return enqueue_spmm(h, X, N, x_scale, Y, static_cast<cudaStream_t>(stream), h->d_acc, h->d_cnt, h->timers_on);
}

// ---- us_spmm_static_scratch: the SpMM with its scratch in a fixed device array ------------------
// The array lives in the library image: every GPU that loads the library holds it until exit.
// In host code `g_static_scratch` is only a stand-in for the symbol; the device address is looked
// up once per device with cudaGetSymbolAddress and that pointer is what the kernel receives.
static __device__ __align__(256) unsigned char g_static_scratch[US_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<void*> g_scratch_addr[kMaxDevices];   // zero-initialised; one look-up per device
}  // namespace

us_status us_spmm_static_scratch(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y,
                                 void* stream)
{
    const us_status s = check_spmm_args(h, X, N, x_scale, Y);
    if (s != US_OK) return s;
    const us::HostMatrix& hm = h->host;
    // scratch the kernel needs: INT32 strip sums, then one arrival counter per strip
    const size_t acc_bytes = (size_t)hm.n_strips * nt_for(N) * 128 * sizeof(int32_t);
    const size_t cnt_bytes = (size_t)hm.n_strips * sizeof(uint32_t);
    if (acc_bytes + cnt_bytes > (size_t)US_STATIC_SCRATCH_BYTES) return US_ERR_SCRATCH_TOO_SMALL;

    const int dev = h->device;   // checked above: it is the current device
    if (dev < 0 || dev >= kMaxDevices) return US_ERR_INVALID_ARG;
    void* ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {  // set-up, once per device, with that device current (threads racing here all
                 // look up the same address)
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) { h->sticky = e; return US_ERR_CUDA; }
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    unsigned char* scratch = static_cast<unsigned char*>(ptr);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps the previous call's contents: sums and counters must start at zero.
    const cudaError_t e = cudaMemsetAsync(scratch, 0, acc_bytes + cnt_bytes, st);
    if (e != cudaSuccess) { h->sticky = e; return US_ERR_CUDA; }
    return enqueue_spmm(h, X, N, x_scale, Y, st, reinterpret_cast<int32_t*>(scratch),
                        reinterpret_cast<uint32_t*>(scratch + acc_bytes), false);
}

// ---- chained calls: fp16 in, INT4 inside, fp16 out ---------------------------------------------
namespace {
cudaError_t launch_quantize(const uint16_t* X16, int64_t ldx, int32_t N, int64_t K, const uint32_t* amax, uint8_t* Xq,
                            uint16_t* x_scale, cudaStream_t st)
{
    const int64_t units = (K + 7) / 8;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::max<int64_t>(1, std::min<int64_t>(64, (units + 255) / 256)), (unsigned)N);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_knob() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, us::us_quantize_f16_kernel, X16, ldx, K, amax, Xq, x_scale);
}
}  // namespace

us_status us_spmm_requant(us_handle* h, const void* X16, int64_t ldx, const void* x_amax, int32_t N, void* Y16,
                          void* y_amax, int64_t amax_m0, int64_t amax_m1, void* stream)
{
    if (!h || !X16 || !x_amax || !Y16 || N < 1 || N > h->max_N) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (!h->d_w_scale) return US_ERR_INVALID_ARG;   // fp16 output needs the weight scales
    if (y_amax && h->host.fmt.C_A != 1) return US_ERR_UNSUPPORTED;   // no absmax-tracking kernel for folded tiles
    if (ldx < h->host.K) return US_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X16) % 2 || reinterpret_cast<uintptr_t>(Y16) % 2 ||
        reinterpret_cast<uintptr_t>(x_amax) % 4 || reinterpret_cast<uintptr_t>(y_amax) % 4) return US_ERR_INVALID_ARG;
    if (y_amax && (amax_m0 < 0 || amax_m1 > h->host.M || amax_m0 > amax_m1)) return US_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return US_ERR_CUDA;
    if (dev != h->device) return US_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (y_amax == x_amax) return US_ERR_INVALID_ARG;
    ChainArgs c;
    c.y_amax = y_amax; c.m0 = amax_m0; c.m1 = amax_m1;
    // One small kernel quantises the activations once into the handle's buffer; it is launched like
    // the SpMM kernels, so the SpMM's weight copies start while it runs. (Quantising inside the SpMM's
    // own staging was measured: every one of the 148 CTAs then pulls the fp16 activations through L2
    // and converts them -- 5 us more than this at N = 1, 8 to 15 us more at N = 16 and 32.)
    uint16_t* xs = reinterpret_cast<uint16_t*>(h->d_xq + h->xq_bytes);
    const cudaError_t e = launch_quantize(static_cast<const uint16_t*>(X16), ldx, N, h->host.K,
                                          static_cast<const uint32_t*>(x_amax), h->d_xq, xs, st);
    if (e != cudaSuccess) { h->sticky = e; return US_ERR_CUDA; }
    return enqueue_spmm(h, h->d_xq, N, xs, Y16, st, h->d_acc, h->d_cnt, h->timers_on, &c);
}

us_status us_absmax_f16(const void* X16, int64_t ldx, int32_t N, int64_t K, void* amax, void* stream)
{
    if (!X16 || !amax || N < 1 || N > 64 || K < 1 || ldx < K) return US_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X16) % 2 || reinterpret_cast<uintptr_t>(amax) % 4) return US_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t units = (K + 7) / 8;
    const unsigned gx = (unsigned)std::max<int64_t>(1, std::min<int64_t>(16, (units + 255) / 256));
    us::us_absmax_f16_kernel<<<dim3(gx, (unsigned)N), 256, 0, st>>>(static_cast<const uint16_t*>(X16), ldx, K, N,
                                                                    static_cast<uint32_t*>(amax));
    if (cudaGetLastError() != cudaSuccess) return US_ERR_CUDA;
    return US_OK;
}

us_status us_quantize_f16(const void* X16, int64_t ldx, int32_t N, int64_t K, const void* amax, void* Xq,
                          void* x_scale, void* stream)
{
    if (!X16 || !amax || !Xq || N < 1 || N > 64 || K < 1 || ldx < K) return US_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X16) % 2 || reinterpret_cast<uintptr_t>(amax) % 4 ||
        reinterpret_cast<uintptr_t>(x_scale) % 2) return US_ERR_INVALID_ARG;
    const cudaError_t e = launch_quantize(static_cast<const uint16_t*>(X16), ldx, N, K, static_cast<const uint32_t*>(amax),
                                          static_cast<uint8_t*>(Xq), static_cast<uint16_t*>(x_scale),
                                          static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { cudaGetLastError(); return US_ERR_CUDA; }
    return US_OK;
}

us_status us_last_error(us_handle* h)
{
    if (!h) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_OK;
    cudaError_t e = cudaDeviceSynchronize();
    uint32_t flag = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&flag, h->d_err, 4, cudaMemcpyDeviceToHost);
    const bool failed = flag != 0 || h->sticky != cudaSuccess || e != cudaSuccess;
    if (failed) {
        // A call that gave up leaves partial sums and arrival counts behind: clear them, so that the
        // next call on this handle starts from the zeroed workspace it relies on.
        cudaMemset(h->d_err, 0, 4);
        cudaMemset(h->d_acc, 0, h->acc_bytes);
        cudaMemset(h->d_cnt, 0, h->cnt_bytes);
        cudaDeviceSynchronize();
    }
    if (h->sticky != cudaSuccess) { e = h->sticky; h->sticky = cudaSuccess; }
    if (e != cudaSuccess) { cudaGetLastError(); return US_ERR_CUDA; }
    if (flag == us::kErrTimeout) return US_ERR_DEVICE_TIMEOUT;
    return flag ? US_ERR_CUDA : US_OK;
}

us_status us_debug_withhold_copy(us_handle* h, int64_t position, int64_t wait_us)
{
    if (!h) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (position < 0) {
        h->withhold = 0xFFFFFFFFu;
        h->wait_ns_hi = 2000000u;
        return US_OK;
    }
    if (position >= h->host.n_items || wait_us < 1 || wait_us > 2000000) return US_ERR_INVALID_ARG;
    h->withhold = (uint32_t)position;
    h->wait_ns_hi = (uint32_t)std::max<int64_t>(1, wait_us * 1000 / 1024);
    return US_OK;
}

us_status us_stage_timers(us_handle* h, int32_t enable, uint64_t* out, int32_t n_out)
{
    if (!h || (out && n_out < 8)) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    const size_t bytes = us::kTimerWords * sizeof(unsigned long long);
    if (!h->d_timers) {
        if (cudaMalloc((void**)&h->d_timers, bytes) != cudaSuccess) return US_ERR_ALLOC;
        cudaMemset(h->d_timers, 0, bytes);
    }
    if (out) {
        if (cudaDeviceSynchronize() != cudaSuccess) return US_ERR_CUDA;
        std::vector<uint64_t> t((size_t)us::kTimerWords);
        if (cudaMemcpy(t.data(), h->d_timers, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return US_ERR_CUDA;
        // reduce the per-warp records
        uint64_t sum[6] = {0, 0, 0, 0, 0, 0}, ck[4] = {0, 0, 0, 0}, max_life = 0, t_min = ~0ull, t_max = 0;
        std::vector<uint64_t> cta((size_t)5 * us::kMaxCtas, 0);   // per CTA: start, first warp end, X staged, end, past the dependency wait
        for (int c = 0; c < us::kMaxCtas; ++c) {
            uint64_t st = ~0ull, first_end = ~0ull, xs = 0, en = 0, pw = 0;
            for (int w = 0; w < us::kMaxWarpsPerCta; ++w) {
                const uint64_t* R = t.data() + (size_t)us::kWarpRec * ((size_t)c * us::kMaxWarpsPerCta + w);
                if (!R[0]) continue;
                for (int i = 0; i < 4; ++i) sum[i] += R[1 + i];
                sum[4] += 1;
                sum[5] += R[5];
                max_life = std::max(max_life, R[4]);
                for (int i = 0; i < 4; ++i) ck[i] += R[9 + i];
                st = std::min(st, R[6]); first_end = std::min(first_end, R[8]); xs = std::max(xs, R[7]);
                en = std::max(en, R[8]); pw = std::max(pw, R[13]);
            }
            if (en) {
                t_min = std::min(t_min, st); t_max = std::max(t_max, en);
                cta[5 * c] = st; cta[5 * c + 1] = first_end; cta[5 * c + 2] = xs; cta[5 * c + 3] = en; cta[5 * c + 4] = pw;
            }
        }
        for (int i = 0; i < 6; ++i) out[i] = sum[i];
        out[6] = max_life;
        out[7] = t_max > t_min ? t_max - t_min : 0;   // first warp start to last warp end, ns
        // optional tail: prologue checkpoints, then five time stamps per CTA
        for (int i = 8; i < n_out; ++i) {
            const int j = i - 8;
            uint64_t v = 0;
            if (j < 4) v = ck[j];
            else if (j - 4 < 5 * us::kMaxCtas) v = cta[j - 4] ? cta[j - 4] - t_min : 0;
            out[i] = v;
        }
        cudaMemset(h->d_timers, 0, bytes);
    }
    if (enable >= 0) h->timers_on = enable != 0;
    return US_OK;
}

us_status us_destroy(us_handle* h)
{
    if (!h) return US_OK;
    if (h->on_device) free_device(h);
    delete h;
    return US_OK;
}

int64_t us_spmm_bytes(const us_handle* h, int32_t N, int32_t fp16_out)
{
    if (!h || N < 1) return -1;
    us_stats st;
    us::fill_stats(h->host, &st);
    const int64_t x = (int64_t)N * ((h->host.K + 1) / 2);
    const int64_t y = (int64_t)N * h->host.M * (fp16_out ? 2 : 4);
    const int64_t sc = fp16_out ? 2 * (h->host.M + N) : 0;
    return st.bytes_total + x + y + sc;
}

const char* us_status_string(us_status s)
{
    switch (s) {
        case US_OK: return "ok";
        case US_ERR_INVALID_ARG: return "invalid argument";
        case US_ERR_VALUE_RANGE: return "weight value outside [-8, 7]";
        case US_ERR_SHAPE: return "format parameters do not fit the tile";
        case US_ERR_UNSUPPORTED: return "format or call not supported";
        case US_ERR_ALLOC: return "allocation failed";
        case US_ERR_CUDA: return "CUDA error";
        case US_ERR_DEVICE_TIMEOUT: return "bounded device wait ran out";
        case US_ERR_SCRATCH_TOO_SMALL: return "problem needs more scratch than the fixed device array holds";
    }
    return "unknown status";
}

}  // extern "C"
