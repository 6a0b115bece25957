// C ABI of the library (declared in include/unionsparse.h): handle management, upload, launch.
#include <algorithm>
#include <cstdio>
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
    uint8_t* d_blob = nullptr;
    uint32_t* d_item_off = nullptr;
    uint32_t* d_cta_begin = nullptr;
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

constexpr int kStages = 2;
constexpr int kMaxWarps = 16;
constexpr int kMinWarps = 2;

int nt_for(int N) { return N <= 8 ? 1 : N <= 16 ? 2 : N <= 32 ? 4 : 8; }

struct LaunchGeom {
    int nt, warps, smem;
    uint32_t slot_bytes;
};

// Shared-memory layout of us_spmm_kernel: selector table, int8 X segment, per-token sums,
// mbarriers, claim counter, then the per-warp rings.
bool plan_launch(const us_handle* h, int N, LaunchGeom* g)
{
    g->nt = nt_for(N);
    g->slot_bytes = (h->host.max_item_bytes + 256u + 127u) & ~127u;
    const int fixed = (int)us::kLutBytes + g->nt * 8 * (h->host.fmt.K_L + 32) + 64 * 4 +
                      32 * kStages * 8 + 32 * 4 + 128;
    const int limit = h->max_smem > 0 ? h->max_smem : 227 * 1024;
    int warps = (limit - fixed) / (int)(kStages * g->slot_bytes);
    warps = std::min(warps, kMaxWarps);
    if (warps < kMinWarps) return false;
    g->warps = warps;
    g->smem = fixed + warps * kStages * (int)g->slot_bytes;
    return true;
}

template <int NT>
cudaError_t launch_nt(const us::SpmmParams& p, int grid, int block, int smem, cudaStream_t st)
{
    if (p.mask_rows % 2 == 0)
        us::us_spmm_kernel<NT, kStages, 2><<<grid, block, smem, st>>>(p);
    else
        us::us_spmm_kernel<NT, kStages, 1><<<grid, block, smem, st>>>(p);
    return cudaGetLastError();
}

// Opt every kernel variant in to the device's full dynamic shared memory (once per handle, at
// encode time, so that us_spmm itself is nothing but a launch).
template <int NT>
cudaError_t enable_large_smem_nt(int bytes)
{
    cudaError_t e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, kStages, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(us::us_spmm_kernel<NT, kStages, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e;
}
cudaError_t enable_large_smem(int bytes)
{
    cudaError_t e = enable_large_smem_nt<1>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_nt<2>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_nt<4>(bytes);
    if (e == cudaSuccess) e = enable_large_smem_nt<8>(bytes);
    return e;
}

void free_device(us_handle* h)
{
    cudaFree(h->d_blob); cudaFree(h->d_item_off); cudaFree(h->d_cta_begin);
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
    if (flags & US_ENCODE_HOST_ONLY) { *out = h; return US_OK; }

    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device);
    if (e == cudaSuccess) e = enable_large_smem(h->max_smem);
    if (e != cudaSuccess) { delete h; return US_ERR_CUDA; }

    const us::HostMatrix& hm = h->host;
    std::vector<uint32_t> sched;
    us::make_schedule(hm, h->sm_count, &sched);
    const int nt_max = nt_for(max_N);
    const size_t acc_bytes = (size_t)hm.n_strips * nt_max * 128 * sizeof(int32_t);
    const size_t cnt_bytes = (size_t)hm.n_strips * sizeof(uint32_t);
    e = upload(&h->d_blob, hm.blob.data(), hm.blob.size());
    if (e == cudaSuccess) e = upload(&h->d_item_off, hm.item_off.data(), hm.item_off.size() * 4);
    if (e == cudaSuccess) e = upload(&h->d_cta_begin, sched.data(), sched.size() * 4);
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
    p.blob = h->d_blob; p.item_off = h->d_item_off; p.cta_begin = h->d_cta_begin;
    p.row_order = h->d_row_order; p.w_scale = h->d_w_scale;
    p.X = static_cast<const uint8_t*>(X);
    p.x_scale = static_cast<const uint16_t*>(x_scale);
    p.Y = Y; p.acc = h->d_acc; p.cnt = h->d_cnt; p.err = h->d_err;
    p.timers = h->timers_on ? h->d_timers : nullptr;
    p.M = (int32_t)hm.M; p.K = (int32_t)hm.K; p.N = N;
    p.n_strips = (int32_t)hm.n_strips; p.n_segs = (int32_t)hm.n_segs;
    p.nkb = hm.nkb; p.mask_rows = hm.mask_rows; p.K_L = hm.fmt.K_L;
    p.slot_bytes = g.slot_bytes;
    p.x_fast = (hm.K % 8 == 0) ? 1 : 0;
    p.fp16_out = x_scale ? 1 : 0;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (g.nt) {
        case 1: e = launch_nt<1>(p, h->sm_count, g.warps * 32, g.smem, st); break;
        case 2: e = launch_nt<2>(p, h->sm_count, g.warps * 32, g.smem, st); break;
        case 4: e = launch_nt<4>(p, h->sm_count, g.warps * 32, g.smem, st); break;
        default: e = launch_nt<8>(p, h->sm_count, g.warps * 32, g.smem, st); break;
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

us_status us_stage_timers(us_handle* h, int32_t enable, uint64_t* out5)
{
    if (!h) return US_ERR_INVALID_ARG;
    if (!h->on_device) return US_ERR_UNSUPPORTED;
    if (!h->d_timers) {
        if (cudaMalloc((void**)&h->d_timers, 8 * sizeof(unsigned long long)) != cudaSuccess) return US_ERR_ALLOC;
        cudaMemset(h->d_timers, 0, 8 * sizeof(unsigned long long));
    }
    if (out5) {
        if (cudaDeviceSynchronize() != cudaSuccess) return US_ERR_CUDA;
        if (cudaMemcpy(out5, h->d_timers, 5 * sizeof(uint64_t), cudaMemcpyDeviceToHost) != cudaSuccess) return US_ERR_CUDA;
        cudaMemset(h->d_timers, 0, 8 * sizeof(unsigned long long));
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
    }
    return "unknown status";
}

}  // extern "C"
