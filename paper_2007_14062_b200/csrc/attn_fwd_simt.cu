// CUDA-core BigBird attention forward (arXiv 2007.14062, Eq. (AT) over the block lists of App. D).
// fp32 arithmetic throughout; the path for fp32 tensors and an independent check for the tensor-core kernel.
//
// One CTA per (batch*head, query block).  Four lanes share a query row, each holding a quarter of the head
// dimension; key blocks are staged through shared memory 32 keys at a time and folded into a running
// (max, sum, output) triple per row (online softmax).
#include <cuda_bf16.h>
#include <math_constants.h>

#include "kernels.h"
#include "../../include/bigbird.h"

namespace bigbird {
namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerRow = 4;
constexpr int kRowsPerPass = kThreads / kLanesPerRow;
constexpr int kKeyChunk = 32;

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_val(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_val(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_fwd_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                     const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                     const uint8_t* __restrict__ kpm, T* __restrict__ out, float* __restrict__ lse,
                     int H, int64_t N, int b, int nb, float scale) {
    constexpr int DL = D / kLanesPerRow;           // head dims per lane: d = sub + 4*i
    __shared__ float sk[kKeyChunk][D];
    __shared__ float sv[kKeyChunk][D];
    __shared__ uint8_t svalid[kKeyChunk];

    const int j = blockIdx.x;
    const int bh = blockIdx.y;
    const int h = bh % H, batch = bh / H;
    const int sub = threadIdx.x % kLanesPerRow;
    const int rloc = threadIdx.x / kLanesPerRow;
    const int64_t base = (int64_t)bh * N * D;
    const int list_begin = row_ptr[(int64_t)h * nb + j], list_end = row_ptr[(int64_t)h * nb + j + 1];
    const uint8_t* mask = kpm ? kpm + (int64_t)batch * N : nullptr;

    for (int r0 = 0; r0 < b; r0 += kRowsPerPass) {
        const int row = r0 + rloc;
        const bool row_ok = row < b;
        const int64_t tok = (int64_t)j * b + row;
        float qr[DL], o[DL];
#pragma unroll
        for (int i = 0; i < DL; ++i) {
            qr[i] = row_ok ? to_float(q[base + tok * D + sub + kLanesPerRow * i]) * scale : 0.f;
            o[i] = 0.f;
        }
        float m = -CUDART_INF_F, l = 0.f;
        for (int e = list_begin; e < list_end; ++e) {
            const int64_t key0 = (int64_t)col_idx[e] * b;
            for (int c0 = 0; c0 < b; c0 += kKeyChunk) {
                const int nk = min(kKeyChunk, b - c0);
                __syncthreads();
                for (int idx = threadIdx.x; idx < nk * D; idx += kThreads) {
                    const int kk = idx / D, d = idx % D;
                    sk[kk][d] = to_float(k[base + (key0 + c0 + kk) * D + d]);
                    sv[kk][d] = to_float(v[base + (key0 + c0 + kk) * D + d]);
                }
                if (threadIdx.x < nk) svalid[threadIdx.x] = mask ? mask[key0 + c0 + threadIdx.x] : (uint8_t)1;
                __syncthreads();
                float s[kKeyChunk];
                float cmax = -CUDART_INF_F;
#pragma unroll
                for (int kk = 0; kk < kKeyChunk; ++kk) {
                    float acc = 0.f;
                    if (kk < nk) {
#pragma unroll
                        for (int i = 0; i < DL; ++i) acc = fmaf(qr[i], sk[kk][sub + kLanesPerRow * i], acc);
                    }
                    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
                    s[kk] = (kk < nk && svalid[kk]) ? acc : -CUDART_INF_F;
                    cmax = fmaxf(cmax, s[kk]);
                }
                if (cmax == -CUDART_INF_F) continue;        // whole chunk masked (uniform across the CTA)
                const float m_new = fmaxf(m, cmax);
                const float alpha = expf(m - m_new);        // m = -inf on the first chunk gives 0
                l *= alpha;
#pragma unroll
                for (int i = 0; i < DL; ++i) o[i] *= alpha;
#pragma unroll
                for (int kk = 0; kk < kKeyChunk; ++kk) {
                    const float p = expf(s[kk] - m_new);    // exp(-inf) = 0 for masked keys
                    l += p;
                    if (kk < nk) {
#pragma unroll
                        for (int i = 0; i < DL; ++i) o[i] = fmaf(p, sv[kk][sub + kLanesPerRow * i], o[i]);
                    }
                }
                m = m_new;
            }
        }
        if (row_ok) {
            const bool q_valid = mask ? mask[tok] != 0 : true;
            const bool any = q_valid && l > 0.f;
            const float inv = any ? 1.f / l : 0.f;
#pragma unroll
            for (int i = 0; i < DL; ++i) store_val(&out[base + tok * D + sub + kLanesPerRow * i], o[i] * inv);
            if (lse && sub == 0) lse[(int64_t)bh * N + tok] = any ? m + logf(l) : -CUDART_INF_F;
        }
    }
}

template <typename T>
cudaError_t launch_t(const FwdArgs& a, const DeviceLayout& dl) {
    dim3 grid((unsigned)a.nb, (unsigned)(a.B * a.H));
    dim3 block(kThreads);
#define BB_LAUNCH(DD)                                                                                     \
    attn_fwd_simt_kernel<T, DD><<<grid, block, 0, a.stream>>>((const T*)a.q, (const T*)a.k, (const T*)a.v, \
        dl.row_ptr, dl.col_idx, a.kpm, (T*)a.out, a.lse, a.H, a.N, a.b, a.nb, a.scale)
    switch (a.D) {
        case 32: BB_LAUNCH(32); break;
        case 64: BB_LAUNCH(64); break;
        case 128: BB_LAUNCH(128); break;
        default: return cudaErrorInvalidValue;
    }
#undef BB_LAUNCH
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_fwd_simt(const FwdArgs& a, const DeviceLayout& dl, int* launches) {
    if ((int64_t)a.B * a.H > 65535) return cudaErrorInvalidValue;
    cudaError_t e = a.dtype == BIGBIRD_BF16 ? launch_t<__nv_bfloat16>(a, dl) : launch_t<float>(a, dl);
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace bigbird
