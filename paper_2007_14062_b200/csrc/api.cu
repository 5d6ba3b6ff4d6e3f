// C-ABI entry points that touch the GPU: argument checks, device copies of the layout, library-owned
// scratch, kernel dispatch.  See include/bigbird.h for the contract of each function.
#include <cuda_runtime.h>

#include <mutex>
#include <new>

#include "kernels.h"
#include "../../include/bigbird.h"

namespace bigbird {
namespace {

thread_local int t_last_cuda_error = 0;
thread_local int t_last_launches = 0;

constexpr int kMaxDevices = 64;
std::mutex g_mu;
DeviceScratch g_scratch[kMaxDevices];

int cuda_fail(cudaError_t e) {
    t_last_cuda_error = (int)e;
    return BIGBIRD_ECUDA;
}

// Library scratch of the current device, created on first use.
int get_scratch(int device, DeviceScratch** out) {
    if (device < 0 || device >= kMaxDevices) return BIGBIRD_EUNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceScratch& s = g_scratch[device];
    if (!s.status) {
        int* p = nullptr;
        cudaError_t e = cudaMalloc(&p, sizeof(int) * (2 + 2 * kCounterSlots));
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaMemset(p, 0, sizeof(int) * (2 + 2 * kCounterSlots));
        if (e != cudaSuccess) { cudaFree(p); return cuda_fail(e); }
        s.status = p;
        s.counters = p + 2;
    }
    *out = &s;
    return BIGBIRD_OK;
}

template <typename T>
cudaError_t upload(T** dst, const void* src, size_t count) {
    *dst = nullptr;
    cudaError_t e = cudaMalloc((void**)dst, (count ? count : 1) * sizeof(T));
    if (e != cudaSuccess || count == 0) return e;
    return cudaMemcpy(*dst, src, count * sizeof(T), cudaMemcpyHostToDevice);
}

void free_device_layout(DeviceLayout& d) {
    cudaFree(d.row_ptr);
    cudaFree(d.col_idx);
    cudaFree(d.col_ptr);
    cudaFree(d.row_idx);
    cudaFree(d.items);
    cudaFree(d.steps);
    cudaFree(d.split_tile_q);
    d = DeviceLayout{};
}

// Device copy of the layout on the current device (made on first use, remade if the device changes).
int get_device_layout(const bigbird_layout* L, int device, DeviceLayout* out) {
    std::lock_guard<std::mutex> lock(L->mu);
    DeviceLayout& d = L->dev;
    if (d.device != device) {
        if (d.device >= 0) {
            int cur = device;
            cudaSetDevice(d.device);
            free_device_layout(d);
            cudaSetDevice(cur);
        }
        cudaError_t e = upload(&d.row_ptr, L->row_ptr.data(), L->row_ptr.size());
        if (e == cudaSuccess) e = upload(&d.col_idx, L->col_idx.data(), L->col_idx.size());
        if (e == cudaSuccess) e = upload(&d.col_ptr, L->col_ptr.data(), L->col_ptr.size());
        if (e == cudaSuccess) e = upload(&d.row_idx, L->row_idx.data(), L->row_idx.size());
        if (e == cudaSuccess) e = upload(&d.items, L->items_abs.data(), L->items_abs.size());
        if (e == cudaSuccess) e = upload(&d.steps, L->steps.data(), L->steps.size());
        if (e == cudaSuccess) e = upload(&d.split_tile_q, L->split_tile_q.data(), L->split_tile_q.size());
        if (e != cudaSuccess) { free_device_layout(d); return cuda_fail(e); }
        d.device = device;
    }
    *out = d;
    return BIGBIRD_OK;
}

int check_common(const void* q, const void* k, const void* v, const bigbird_layout* L, void* out,
                 int B, int H, int64_t N, int D, int b, int dtype) {
    if (!q || !k || !v || !L || !out) return BIGBIRD_EINVAL;
    if (B < 1 || H < 1 || N < 1 || D < 1 || b < 1) return BIGBIRD_EINVAL;
    if (L->N != N || L->b != b || L->H != H) return BIGBIRD_EINVAL;
    if (dtype != BIGBIRD_FP32 && dtype != BIGBIRD_BF16) return BIGBIRD_EUNSUPPORTED;
    if ((((uintptr_t)q) | ((uintptr_t)k) | ((uintptr_t)v) | ((uintptr_t)out)) & 15) return BIGBIRD_EINVAL;
    return BIGBIRD_OK;
}

int fwd(bool force_simt, const void* q, const void* k, const void* v, const bigbird_layout* L,
        const uint8_t* kpm, void* out, float* lse, int B, int H, int64_t N, int D, int b, float scale,
        int dtype, void* stream) {
    t_last_launches = 0;
    int rc = check_common(q, k, v, L, out, B, H, N, D, b, dtype);
    if (rc != BIGBIRD_OK) return rc;
    const bool simt = force_simt || dtype == BIGBIRD_FP32;
    if (simt) {
        if (D != 32 && D != 64 && D != 128) return BIGBIRD_EUNSUPPORTED;
        if ((int64_t)B * H > 65535) return BIGBIRD_EUNSUPPORTED;
    } else {
        if (D != 64 || b != 64) return BIGBIRD_EUNSUPPORTED;
    }
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
    DeviceLayout dl;
    rc = get_device_layout(L, device, &dl);
    if (rc != BIGBIRD_OK) return rc;
    FwdArgs a{q, k, v, kpm, out, lse, B, H, D, b, L->nb, N, scale, dtype, (cudaStream_t)stream};
    if (simt) {
        e = launch_attn_fwd_simt(a, dl, &t_last_launches);
        return e == cudaSuccess ? BIGBIRD_OK : cuda_fail(e);
    }
    DeviceScratch* sc = nullptr;
    rc = get_scratch(device, &sc);
    if (rc != BIGBIRD_OK) return rc;
    cudaError_t ce = cudaSuccess;
    rc = launch_attn_fwd_sm100(a, *L, dl, *sc, &t_last_launches, &ce);
    if (rc == BIGBIRD_ECUDA) t_last_cuda_error = (int)ce;
    return rc;
}

}  // namespace
}  // namespace bigbird

extern "C" {

int bigbird_attn_fwd(const void* q, const void* k, const void* v, const bigbird_layout* layout,
                     const uint8_t* key_padding_mask, void* out, float* lse, int B, int H, int64_t N, int D,
                     int b, float scale, int dtype, void* stream) {
    return bigbird::fwd(false, q, k, v, layout, key_padding_mask, out, lse, B, H, N, D, b, scale, dtype, stream);
}

int bigbird_attn_fwd_simt(const void* q, const void* k, const void* v, const bigbird_layout* layout,
                          const uint8_t* key_padding_mask, void* out, float* lse, int B, int H, int64_t N,
                          int D, int b, float scale, int dtype, void* stream) {
    return bigbird::fwd(true, q, k, v, layout, key_padding_mask, out, lse, B, H, N, D, b, scale, dtype, stream);
}

int bigbird_attn_bwd(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                     const bigbird_layout* layout, const uint8_t* key_padding_mask, void* dq, void* dk, void* dv,
                     int B, int H, int64_t N, int D, int b, float scale, int dtype, void* stream) {
    using namespace bigbird;
    t_last_launches = 0;
    int rc = check_common(q, k, v, layout, dq, B, H, N, D, b, dtype);
    if (rc != BIGBIRD_OK) return rc;
    if (!out || !lse || !dout || !dk || !dv) return BIGBIRD_EINVAL;
    if ((((uintptr_t)out) | ((uintptr_t)dout) | ((uintptr_t)dk) | ((uintptr_t)dv)) & 15) return BIGBIRD_EINVAL;
    if (D != 32 && D != 64 && D != 128) return BIGBIRD_EUNSUPPORTED;
    if ((int64_t)B * H > 65535) return BIGBIRD_EUNSUPPORTED;
    if (!(scale > 0.f) || !(scale < INFINITY)) return BIGBIRD_EINVAL;
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
    DeviceLayout dl;
    rc = get_device_layout(layout, device, &dl);
    if (rc != BIGBIRD_OK) return rc;
    BwdArgs a{q, k, v, out, lse, dout, key_padding_mask, dq, dk, dv, B, H, D, b, layout->nb, N, scale, dtype, (cudaStream_t)stream};
    e = launch_attn_bwd_simt(a, dl, &t_last_launches);
    return e == cudaSuccess ? BIGBIRD_OK : cuda_fail(e);
}

int bigbird_layout_destroy(bigbird_layout* L) {
    if (!L) return BIGBIRD_EINVAL;
    if (L->dev.device >= 0) {
        int cur = 0;
        const bool have = cudaGetDevice(&cur) == cudaSuccess;
        if (cudaSetDevice(L->dev.device) == cudaSuccess) bigbird::free_device_layout(L->dev);
        if (have) cudaSetDevice(cur);
    }
    delete L;
    return BIGBIRD_OK;
}

int bigbird_last_status(void* stream, int* status, int* detail) {
    if (!status) return BIGBIRD_EINVAL;
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return bigbird::cuda_fail(e);
    bigbird::DeviceScratch* sc = nullptr;
    int rc = bigbird::get_scratch(device, &sc);
    if (rc != BIGBIRD_OK) return rc;
    e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return bigbird::cuda_fail(e);
    int host[2] = {0, 0};
    e = cudaMemcpy(host, sc->status, sizeof(host), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return bigbird::cuda_fail(e);
    if (host[0] != 0) {
        // a kernel gave up: its work counters may be left non-zero, so clear the whole block
        e = cudaMemset(sc->status, 0, sizeof(int) * (2 + 2 * bigbird::kCounterSlots));
        if (e != cudaSuccess) return bigbird::cuda_fail(e);
    }
    *status = host[0];
    if (detail) *detail = host[1];
    return BIGBIRD_OK;
}

int bigbird_selftest_wait_expiry(void* stream) {
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return bigbird::cuda_fail(e);
    bigbird::DeviceScratch* sc = nullptr;
    int rc = bigbird::get_scratch(device, &sc);
    if (rc != BIGBIRD_OK) return rc;
    e = bigbird::launch_wait_expiry_selftest(*sc, (cudaStream_t)stream);
    return e == cudaSuccess ? BIGBIRD_OK : bigbird::cuda_fail(e);
}

int bigbird_last_cuda_error(void) { return bigbird::t_last_cuda_error; }
int bigbird_last_launch_count(void) { return bigbird::t_last_launches; }

}  // extern "C"
