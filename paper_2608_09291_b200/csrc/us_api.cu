// C ABI of the library (declared in include/unionsparse.h): handle management, upload, launch.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "us_host.h"
#include "us_spmm_kernel.cuh"

struct us_handle {
    us::HostMatrix host;
    bool on_device = false;
    int device = -1;
    int sm_count = 0;
    int max_N = 0;
    int max_smem = 0;
    int co_warps = 10;   // warps of an N <= 8 CTA when two CTAs share an SM's registers
    int co_warps2 = 8;   // the same for the N = 9..16 kernel with packed activations
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
    unsigned long long* d_timers = nullptr;
    bool timers_on = false;
    cudaError_t sticky = cudaSuccess;
};

namespace {

constexpr int kMinWarps = 2;

int nt_for(int N) { return N <= 8 ? 1 : N <= 16 ? 2 : N <= 32 ? 4 : 8; }
int class_of(int nt) { return nt == 1 ? 0 : nt == 2 ? 1 : nt == 4 ? 2 : 3; }

// Tuning knobs, overridable from the environment (read once per process) for experiments.
int env_int(const char* name, int fallback)
{
    const char* v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : fallback;
}
int x_budget() { static int v = env_int("US_X_BUDGET_KB", 0) * 1024; return v; }           // int8 X of one K range; 0 = automatic
int local_acc_budget() { static int v = env_int("US_LOCAL_ACC_KB", 32) * 1024; return v; }  // local strip sums
int stages_knob() { static int v = env_int("US_STAGES", 0); return v; }     // ring slots per warp, 0 = automatic
int lut_rep_knob() { static int v = env_int("US_LUT_REP", 0); return v; }   // selector-table copies, 0 = automatic
int pdl_knob() { static int v = env_int("US_PDL", 1); return v; }          // programmatic dependent launch
int coresident_tiles_knob() { static int v = env_int("US_CORESIDENT_TILES", 16); return v; }
int local_acc_cap() { static int v = env_int("US_LOCAL_ACC_CAP_KB", 48) * 1024; return v; }
int coresident_knob() { static int v = env_int("US_CORESIDENT", 1); return v; }  // small problems: half an SM per CTA
int max_warps() { static int v = std::min(16, std::max(2, env_int("US_MAX_WARPS", 16))); return v; }

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
int xp_knob() { static int v = env_int("US_PACKED_X", 1); return v; }   // 0 off, 1 automatic, 2 whenever possible
bool plan_debug() { static int v = env_int("US_PLAN_DEBUG", 0); return v != 0; }
int min_warps_knob() { static int v = env_int("US_MIN_WARPS", 12); return v; }
// Shared memory of one K range's activations: int8 (one byte per token and k, 32 bytes of pad per
// token row) or packed (half of that).
int64_t x_bytes(int nt, int64_t G, int K_L, bool xp)
{
    return xp ? (int64_t)nt * 8 * (G * K_L / 2 + 16) : (int64_t)nt * 8 * (G * K_L + 32);
}

int segs_per_range(const us::HostMatrix& hm, int nt, int limit, int64_t min_ranges, bool xp)
{
    const int64_t n_segs = hm.n_segs;
    if (x_budget() > 0) {
        const int g = (x_budget() / (nt * 8) - 32) / hm.fmt.K_L;
        return (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(g, n_segs), (n_segs + min_ranges - 1) / min_ranges));
    }
    const int slot = (int)((hm.max_item_bytes + 256u + 127u) & ~127u);
    const int acc = nt * 512 * 2 <= local_acc_budget() ? local_acc_budget() : 0;
    const int other = 256 * 8 * 4 + (int)us::kLutScratchBytes + acc + 2 * us::kOffTable * 4 + 1024;
    for (int64_t r = std::max<int64_t>(1, min_ranges); r <= n_segs; ++r) {
        // A single range is worth more (no partial sums leave the CTA when the cuts fall on strip
        // boundaries): it may cost two more warps. Measured on 4096 x 11008, N = 8: one range with
        // 15 warps 9.8 us, two ranges with 16 warps 14.7 us.
        const int want = std::min(max_warps(), r == 1 ? std::min(10, min_warps_knob()) : min_warps_knob());
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
    g->slot_bytes = (h->host.max_item_bytes + 256u + 127u) & ~127u;
    // selector table copies: 32 (conflict-free lookups) when that costs no warp, else 8
    int lut_rep = 32;
    auto fixed_for = [&](int rep) {
        return 256 * rep * 4 + (int)us::kLutScratchBytes + (int)x_bytes(g->nt, G, h->host.fmt.K_L, g->xp) + G * g->nt * 8 * 4 +
                           32 * 4 + s_local * (g->nt * 128 + 1) * 4 + 2 * us::kOffTable * 4 + 128;
    };
    int fixed_base = fixed_for(lut_rep);
    const int limit = h->max_smem > 0 ? h->max_smem : 227 * 1024;
    // Ring depth: two slots per warp when that still gives (nearly) all the warps; else one slot per
    // warp and more warps -- measured on the 70B-shaped FFN: 16 warps x 1 slot beat 9 warps x 2.
    auto warps_for = [&](int stages) {
        const int fixed = fixed_base + 32 * stages * 8;
        return std::min((limit - fixed) / (int)(stages * g->slot_bytes), max_warps());
    };
    {
        const int w32 = std::max(warps_for(1), warps_for(2));
        fixed_base = fixed_for(8);
        const int w8 = std::max(warps_for(1), warps_for(2));
        // 32 copies only for long-running CTAs (measured: 1 % faster on the 70B-shaped FFN, but the
        // 4096 x 4096 case -- about one tile per warp -- loses 5 % to the bigger table)
        const bool long_run = (h->host.n_items + 147) / 148 >= 4 * (int64_t)w8;
        if (w32 >= w8 && long_run) { lut_rep = 32; fixed_base = fixed_for(32); } else { lut_rep = 8; }
        if (lut_rep_knob() == 8 || lut_rep_knob() == 32) { lut_rep = lut_rep_knob(); fixed_base = fixed_for(lut_rep); }
    }
    int stages = stages_knob() > 0 ? stages_knob() : (warps_for(1) >= warps_for(2) + 3 ? 1 : 2);
    int warps = warps_for(stages);
    if (warps < kMinWarps) return false;
    // Small problems at N <= 8 (a CTA sees about a tile per warp): take at most half an SM -- shared
    // memory and registers -- with one slot per warp, so that the next launch's CTA moves in beside
    // this one and runs its latency-bound prologue (parameters, offsets, first tile copies, table)
    // under this one's work; with one CTA per SM, programmatic dependent launch alone hides only the
    // launch latency, because all CTAs of a launch end at about the same time.
    // Measured on 4096 x 4096, N = 8: 6.6 -> 5.7 us; not worth it from ~20 tiles per CTA on.
    const int64_t per_cta = (h->host.n_items + 147) / 148;
    int fixed = fixed_base + 32 * stages * 8;
    // (N = 9..16 too, where the plan stages X packed and in local mode: that kernel is as lean.)
    // (Tried at N = 32 as well: 8 warps per CTA, slower.)
    const bool co_class = g->nt == 1 || (g->nt == 2 && g->xp && s_local > 0);
    if (coresident_knob() && co_class && per_cta <= coresident_tiles_knob() && stages_knob() == 0 && lut_rep_knob() == 0) {
        const int half = 228 * 1024 / 2 - 1024 - 512;   // per SM: 228 KB, 1 KB reserved per CTA
        const int fixed8 = fixed_for(8) + 32 * 8;
        int w = std::min(g->nt == 1 ? h->co_warps : h->co_warps2, max_warps());
        while (w >= 8 && fixed8 + w * (int)g->slot_bytes > half) --w;
        if (w >= 8) { stages = 1; lut_rep = 8; warps = w; fixed = fixed8; }
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
                    if (plan_debug())
                        fprintf(stderr, "[unionsparse] plan nt=%d%s: G=%d needs %d local strips\n", nt, xp ? " packed X" : "", G, worst);
                    if (pass == 0 && need <= local_acc_budget()) { *s_local = worst; return G; }
                    if (pass == 1 && need <= local_acc_cap()) {
                        const int slot = (int)((h->host.max_item_bytes + 256u + 127u) & ~127u);
                        const int64_t fixed = 256 * 8 * 4 + (int64_t)us::kLutScratchBytes + need + 2 * us::kOffTable * 4 + 1024 +
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
        if (nt <= 4 && xp_knob() != 0) {
            const int64_t n_segs = h->host.n_segs;
            const int64_t ranges = h->s_local[c] > 0 ? (n_segs + h->G[c] - 1) / h->G[c] : n_segs + 1;
            const bool small_share = nt >= 2 && (int64_t)h->host.blob.size() / std::max(1, n_cta) < 128 * 1024;
            if (ranges > 1 || small_share || xp_knob() == 2) {
                std::vector<uint32_t> alt;
                int sl2 = 0;
                const int G2 = local_plan(true, &alt, &sl2);
                const int64_t ranges2 = G2 > 0 ? (n_segs + G2 - 1) / G2 : 0;
                // (N = 32, packed against plain: 11008 x 4096 21.4 -> 18.5 us, 13824 x 5120 24.9 -> 23.6 us,
                // 5120 x 5120 17.3 -> 18.2 us with one range; three ranges instead of eleven one-segment
                // ranges on 4096 x 11008 were slower, 19.3 -> 26.4 us: only a single range pays)
                if (G2 > 0 && (ranges2 == 1 || xp_knob() == 2)) {
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

int run_knob() { static int v = env_int("US_RUN", 0); return v; }
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
    if (NT <= 4 && xp && la) {   // packed X: planned for these classes and local mode only
        constexpr int NP = NT <= 4 ? NT : 4;
        return timed ? cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NP, ST, true, true, true>, p)
                     : cudaLaunchKernelEx(&cfg, us::us_spmm_kernel<NP, ST, true, false, true>, p);
    }
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
    cudaFree(h->d_cnt); cudaFree(h->d_err); cudaFree(h->d_timers);
}

template <class T>
cudaError_t upload(T** dst, const void* src, size_t bytes)
{
    cudaError_t e = cudaMalloc((void**)dst, std::max<size_t>(bytes, 16));
    if (e != cudaSuccess) return e;
    return bytes ? cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) : cudaSuccess;
}

}  // namespace

extern "C" {

us_status us_encode(const int8_t* W, int64_t M, int64_t K, const uint16_t* w_scale,
                    const us_format* fmt, int32_t max_N, uint32_t flags, us_handle** out)
{
    if (out) *out = nullptr;
    if (!W || !out || M <= 0 || K <= 0 || max_N < 1 || max_N > 64) return US_ERR_INVALID_ARG;
    if (M > 0x7FFFFFF0ll || K > 0x7FFFFFF0ll) return US_ERR_INVALID_ARG;
    us_format f = fmt ? *fmt : us_format{16, us::default_K_L(M, K), 2, 1};
    us_handle* h = new (std::nothrow) us_handle();
    if (!h) return US_ERR_ALLOC;
    h->max_N = max_N;
    us_status s;
    try {
        s = us::encode_host(W, M, K, w_scale, f, flags, 0, &h->host);
    } catch (const std::bad_alloc&) {
        s = US_ERR_ALLOC;
    }
    if (s != US_OK) { delete h; return s; }
    if (h->host.n_items >= (1 << 24) || h->host.n_strips * h->host.n_segs >= (1 << 24) || h->host.n_segs >= (1 << 16)) {
        delete h;
        return US_ERR_UNSUPPORTED;  // the kernel's index arithmetic assumes fewer tiles
    }
    if (flags & US_ENCODE_HOST_ONLY) {
        std::vector<uint32_t> sched[4];
        plan_classes(h, 148, sched);
        *out = h;
        return US_OK;
    }

    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device);
    if (e == cudaSuccess && h->sm_count > us::kMaxCtas) h->sm_count = us::kMaxCtas;
    if (e == cudaSuccess) e = enable_large_smem(h->max_smem);
    if (e == cudaSuccess) {
        // Two N <= 8 CTAs share the SM's 64 K registers (allocated 8 per thread at a time).
        int regs = 0;
        // (the stage-timer builds need more and simply do not share an SM)
        for (const void* f : {(const void*)us::us_spmm_kernel<1, 1, true, false>, (const void*)us::us_spmm_kernel<1, 1, false, false>}) {
            cudaFuncAttributes fa;
            e = cudaFuncGetAttributes(&fa, f);
            if (e != cudaSuccess) break;
            regs = std::max(regs, fa.numRegs);
        }
        if (e == cudaSuccess) h->co_warps = 32768 / (32 * ((regs + 7) / 8 * 8));
        cudaFuncAttributes fa2;
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa2, (const void*)us::us_spmm_kernel<2, 1, true, false, true>);
        if (e == cudaSuccess) h->co_warps2 = 32768 / (32 * ((fa2.numRegs + 7) / 8 * 8));

    }
    if (e != cudaSuccess) { delete h; return US_ERR_CUDA; }

    const us::HostMatrix& hm = h->host;
    std::vector<uint32_t> sched[4];
    plan_classes(h, h->sm_count, sched);
    const int nt_max = nt_for(max_N);
    const size_t acc_bytes = (size_t)hm.n_strips * nt_max * 128 * sizeof(int32_t);
    const size_t cnt_bytes = (size_t)hm.n_strips * sizeof(uint32_t);
    e = upload(&h->d_blob, hm.blob.data(), hm.blob.size());
    if (e == cudaSuccess) e = upload(&h->d_item_off, hm.item_off.data(), hm.item_off.size() * 4);
    for (int c = 0; c < 4; ++c) h->cta_begin[c] = sched[c];
    if (e == cudaSuccess) e = upload(&h->d_row_order, hm.row_order.data(), hm.row_order.size() * 4);
    if (e == cudaSuccess && !hm.w_scale.empty()) e = upload(&h->d_w_scale, hm.w_scale.data(), hm.w_scale.size() * 2);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_acc, acc_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->d_acc, 0, acc_bytes);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_cnt, cnt_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->d_cnt, 0, cnt_bytes);
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
    std::memcpy(perm_out, h->host.row_order.data(), h->host.row_order.size() * sizeof(int32_t));
    return US_OK;
}

us_status us_launch_info(const us_handle* h, int32_t N, int32_t* grid, int32_t* block,
                         int32_t* smem_bytes)
{
    if (!h || N < 1 || N > h->max_N) return US_ERR_INVALID_ARG;
    LaunchGeom g;
    if (!plan_launch(h, N, &g)) return US_ERR_UNSUPPORTED;
    if (grid) *grid = h->sm_count > 0 ? h->sm_count : 148;
    if (block) *block = g.warps * 32;
    if (smem_bytes) *smem_bytes = g.smem;
    return US_OK;
}

us_status us_spmm(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y, void* stream)
{
    if (!h || !X || !Y || N < 1 || N > h->max_N) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (x_scale && !h->d_w_scale) return US_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X) % 16) return US_ERR_INVALID_ARG;
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
        const int want = run_knob() > 0 ? run_knob() : std::min(p.G, 2 * balanced);
        p.run_len = std::max(1, std::min(want, p.G));
    }
    p.row_order = h->d_row_order; p.w_scale = h->d_w_scale;
    p.X = static_cast<const uint8_t*>(X);
    p.x_scale = static_cast<const uint16_t*>(x_scale);
    p.Y = Y; p.acc = h->d_acc; p.cnt = h->d_cnt; p.err = h->d_err;
    p.timers = h->timers_on ? h->d_timers : nullptr;
    p.M = (int32_t)hm.M; p.K = (int32_t)hm.K; p.N = N;
    p.n_strips = (int32_t)hm.n_strips; p.n_segs = (int32_t)hm.n_segs;
    p.nkb = hm.nkb; p.mask_rows = hm.mask_rows; p.K_L = hm.fmt.K_L;
    p.slot_bytes = g.slot_bytes;
    p.x_fast = (hm.K % 32 == 0) ? 2 : (hm.K % 8 == 0) ? 1 : 0;
    p.fp16_out = x_scale ? 1 : 0;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
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

// ---- us_spmm_static_scratch: the SpMM with its scratch in a fixed device array ------------------
// The array lives in the library image: every GPU that loads the library holds it until exit.
// In host code `g_static_scratch` is only a stand-in for the symbol; the device address is looked
// up once per device with cudaGetSymbolAddress and that pointer is what the kernel receives.
static __device__ __align__(256) unsigned char g_static_scratch[US_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};
}  // namespace

us_status us_spmm_static_scratch(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y,
                                 void* stream)
{
    if (!h || !X || !Y || N < 1 || N > h->max_N) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (x_scale && !h->d_w_scale) return US_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X) % 16) return US_ERR_INVALID_ARG;
    LaunchGeom g;
    if (!plan_launch(h, N, &g)) return US_ERR_UNSUPPORTED;

    const us::HostMatrix& hm = h->host;
    // scratch the kernel needs: INT32 strip sums, then one arrival counter per strip
    const size_t acc_bytes = (size_t)hm.n_strips * g.nt * 128 * sizeof(int32_t);
    const size_t cnt_bytes = (size_t)hm.n_strips * sizeof(uint32_t);
    if (acc_bytes + cnt_bytes > (size_t)US_STATIC_SCRATCH_BYTES) return US_ERR_SCRATCH_TOO_SMALL;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return US_ERR_CUDA;
    if (dev != h->device || dev < 0 || dev >= kMaxDevices) return US_ERR_INVALID_ARG;
    if (!g_scratch_addr[dev]) {  // set-up, once per device, with that device current
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) { h->sticky = e; return US_ERR_CUDA; }
        g_scratch_addr[dev] = ptr;
    }
    unsigned char* scratch = static_cast<unsigned char*>(g_scratch_addr[dev]);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps the previous call's contents: sums and counters must start at zero.
    cudaError_t e = cudaMemsetAsync(scratch, 0, acc_bytes + cnt_bytes, st);
    if (e != cudaSuccess) { h->sticky = e; return US_ERR_CUDA; }

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
        const int64_t per_cta = std::max<int64_t>(1, hm.n_items / std::max(1, h->sm_count));
        const int balanced = (int)std::max<int64_t>(1, per_cta / (4 * (int64_t)g.warps));
        const int want = run_knob() > 0 ? run_knob() : std::min(p.G, 2 * balanced);
        p.run_len = std::max(1, std::min(want, p.G));
    }
    p.row_order = h->d_row_order; p.w_scale = h->d_w_scale;
    p.X = static_cast<const uint8_t*>(X);
    p.x_scale = static_cast<const uint16_t*>(x_scale);
    p.Y = Y;
    p.acc = reinterpret_cast<int32_t*>(scratch);
    p.cnt = reinterpret_cast<uint32_t*>(scratch + acc_bytes);
    p.err = h->d_err;
    p.timers = nullptr;
    p.M = (int32_t)hm.M; p.K = (int32_t)hm.K; p.N = N;
    p.n_strips = (int32_t)hm.n_strips; p.n_segs = (int32_t)hm.n_segs;
    p.nkb = hm.nkb; p.mask_rows = hm.mask_rows; p.K_L = hm.fmt.K_L;
    p.slot_bytes = g.slot_bytes;
    p.x_fast = (hm.K % 32 == 0) ? 2 : (hm.K % 8 == 0) ? 1 : 0;
    p.fp16_out = x_scale ? 1 : 0;
    switch (g.nt) {
        case 1: e = launch_nt<1>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
        case 2: e = launch_nt<2>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
        case 4: e = launch_nt<4>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
        default: e = launch_nt<8>(p, g.xp, g.stages, h->sm_count, g.warps * 32, g.smem, st); break;
    }
    if (e != cudaSuccess) { h->sticky = e; return US_ERR_CUDA; }
    return US_OK;
}

us_status us_last_error(us_handle* h)
{
    if (!h) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_OK;
    cudaError_t e = cudaDeviceSynchronize();
    uint32_t flag = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&flag, h->d_err, 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && flag) cudaMemset(h->d_err, 0, 4);
    if (h->sticky != cudaSuccess) { e = h->sticky; h->sticky = cudaSuccess; }
    if (e != cudaSuccess) return US_ERR_CUDA;
    if (flag == us::kErrTimeout) return US_ERR_DEVICE_TIMEOUT;
    return flag ? US_ERR_CUDA : US_OK;
}

static cudaError_t reset_timers(unsigned long long* d)
{
    static unsigned long long z[16 + 4 * us::kMaxCtas];
    std::memset(z, 0, sizeof(z));
    z[7] = ~0ull;  // running minimum of the start time stamps
    return cudaMemcpy(d, z, sizeof(z), cudaMemcpyHostToDevice);
}

us_status us_stage_timers(us_handle* h, int32_t enable, uint64_t* out8)
{
    if (!h) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (!h->d_timers) {
        if (cudaMalloc((void**)&h->d_timers, (16 + 4 * us::kMaxCtas) * sizeof(unsigned long long)) != cudaSuccess) return US_ERR_ALLOC;
        reset_timers(h->d_timers);
    }
    if (out8) {
        if (cudaDeviceSynchronize() != cudaSuccess) return US_ERR_CUDA;
        static uint64_t t[16 + 4 * us::kMaxCtas];
        if (cudaMemcpy(t, h->d_timers, sizeof(t), cudaMemcpyDeviceToHost) != cudaSuccess) return US_ERR_CUDA;
        if (const char* path = std::getenv("US_TIMER_DUMP")) {
            if (FILE* f = std::fopen(path, "a")) {
                for (int c = 0; c < us::kMaxCtas; ++c)
                    if (t[16 + 4 * c])
                        std::fprintf(f, "%d %llu %llu %llu %lld\n", c, (unsigned long long)t[16 + 4 * c], (unsigned long long)t[17 + 4 * c],
                                     (unsigned long long)t[18 + 4 * c], (long long)(t[19 + 4 * c] - t[7]));
                std::fprintf(f, "#\n");
                std::fclose(f);
            }
        }
        for (int i = 0; i < 7; ++i) out8[i] = t[i];
        out8[7] = t[8] > t[7] ? t[8] - t[7] : 0;   // first warp start to last warp end, ns
        if (std::getenv("US_TIMER_DEBUG") && t[4])
            std::fprintf(stderr, "[us] prologue checkpoints (cycles/warp): range known %.0f, copies issued %.0f, table done %.0f, X staged %.0f\n",
                         (double)t[9] / t[4], (double)t[10] / t[4], (double)t[11] / t[4], (double)t[12] / t[4]);
        reset_timers(h->d_timers);
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
