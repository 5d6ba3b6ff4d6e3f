// CUDA-core gradients of BigBird attention (arXiv 2007.14062, Eq. (AT) over the block lists of App. D; the paper
// trains through this op, Sec. 4 and App. E.1, and leaves the derivatives to autodiff).  fp32 arithmetic throughout.
//
// With P = softmax(scale q k^T) over the attended valid keys (recomputed here from the saved lse), out = P v and
// delta_i = sum_d dout[i, d] out[i, d]:
//     dv = P^T dout,   dS = P o (dout v^T - delta),   dq = scale dS k,   dk = scale dS^T q.
// Two kernels: dq by query block over its key-block list, dk and dv by key block over the transposed list (the
// query blocks that attend it).  Four lanes share a query row (first kernel) or a key (second kernel), each holding a
// quarter of the head dimension; the other side is staged through shared memory 32 rows at a time.  Padded query
// rows get dq = 0 and give nothing to dk, dv; padded keys get dk = dv = 0.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "kernels.h"
#include "../../include/bigbird.h"

namespace bigbird {
namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerRow = 4;
constexpr int kRowsPerPass = kThreads / kLanesPerRow;
constexpr int kChunk = 32;

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_val(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_val(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
__device__ __forceinline__ float quad_sum(float x) {
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    return x;
}

// dq[i] = scale * sum_k dS[i, k] k_k for the rows of one query block.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_bwd_dq_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ out,
                   const float* __restrict__ lse, const T* __restrict__ dout, const int32_t* __restrict__ row_ptr,
                   const int32_t* __restrict__ col_idx, const uint8_t* __restrict__ kpm, T* __restrict__ dq,
                   int H, int64_t N, int b, int nb, float scale) {
    constexpr int DL = D / kLanesPerRow;           // head dims per lane: d = sub + 4*i
    __shared__ float sk[kChunk][D];
    __shared__ float sv[kChunk][D];
    __shared__ uint8_t svalid[kChunk];

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
        float qr[DL], dor[DL], acc[DL];
        float delta = 0.f;
#pragma unroll
        for (int i = 0; i < DL; ++i) {
            const int64_t at = base + tok * D + sub + kLanesPerRow * i;
            qr[i] = row_ok ? to_float(q[at]) : 0.f;
            dor[i] = row_ok ? to_float(dout[at]) : 0.f;
            delta = fmaf(dor[i], row_ok ? to_float(out[at]) : 0.f, delta);
            acc[i] = 0.f;
        }
        delta = quad_sum(delta);
        const float my_lse = row_ok ? lse[(int64_t)bh * N + tok] : -CUDART_INF_F;
        // a padded query row, or one without any attended valid key, has no probabilities
        const bool live = row_ok && (mask ? mask[tok] != 0 : true) && my_lse > -CUDART_INF_F;
        for (int e = list_begin; e < list_end; ++e) {
            const int64_t key0 = (int64_t)col_idx[e] * b;
            for (int c0 = 0; c0 < b; c0 += kChunk) {
                const int nk = min(kChunk, b - c0);
                __syncthreads();
                for (int idx = threadIdx.x; idx < nk * D; idx += kThreads) {
                    const int kk = idx / D, d = idx % D;
                    sk[kk][d] = to_float(k[base + (key0 + c0 + kk) * D + d]);
                    sv[kk][d] = to_float(v[base + (key0 + c0 + kk) * D + d]);
                }
                if (threadIdx.x < nk) svalid[threadIdx.x] = mask ? mask[key0 + c0 + threadIdx.x] : (uint8_t)1;
                __syncthreads();
                for (int kk = 0; kk < nk; ++kk) {
                    float s = 0.f, dp = 0.f;
#pragma unroll
                    for (int i = 0; i < DL; ++i) {
                        s = fmaf(qr[i], sk[kk][sub + kLanesPerRow * i], s);
                        dp = fmaf(dor[i], sv[kk][sub + kLanesPerRow * i], dp);
                    }
                    s = quad_sum(s);
                    dp = quad_sum(dp);
                    const float p = (live && svalid[kk]) ? expf(s * scale - my_lse) : 0.f;
                    const float ds = p * (dp - delta);
#pragma unroll
                    for (int i = 0; i < DL; ++i) acc[i] = fmaf(ds, sk[kk][sub + kLanesPerRow * i], acc[i]);
                }
            }
        }
        if (row_ok) {
#pragma unroll
            for (int i = 0; i < DL; ++i) store_val(&dq[base + tok * D + sub + kLanesPerRow * i], acc[i] * scale);
        }
    }
}

// dk[k] = scale * sum_i dS[i, k] q_i and dv[k] = sum_i P[i, k] dout_i for the keys of one key block, over the query
// blocks that attend it.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_bwd_dkv_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ out,
                    const float* __restrict__ lse, const T* __restrict__ dout, const int32_t* __restrict__ col_ptr,
                    const int32_t* __restrict__ row_idx, const uint8_t* __restrict__ kpm, T* __restrict__ dk, T* __restrict__ dv,
                    int H, int64_t N, int b, int nb, float scale) {
    constexpr int DL = D / kLanesPerRow;
    __shared__ float sq[kChunk][D];
    __shared__ float sdo[kChunk][D];
    __shared__ float slse[kChunk];
    __shared__ float sdelta[kChunk];
    __shared__ uint8_t slive[kChunk];

    const int c = blockIdx.x;
    const int bh = blockIdx.y;
    const int h = bh % H, batch = bh / H;
    const int sub = threadIdx.x % kLanesPerRow;
    const int rloc = threadIdx.x / kLanesPerRow;
    const int64_t base = (int64_t)bh * N * D;
    const int list_begin = col_ptr[(int64_t)h * nb + c], list_end = col_ptr[(int64_t)h * nb + c + 1];
    const uint8_t* mask = kpm ? kpm + (int64_t)batch * N : nullptr;

    for (int r0 = 0; r0 < b; r0 += kRowsPerPass) {
        const int key = r0 + rloc;
        const bool key_ok = key < b;
        const int64_t tok = (int64_t)c * b + key;
        const bool key_live = key_ok && (mask ? mask[tok] != 0 : true);
        float kr[DL], vr[DL], adk[DL], adv[DL];
#pragma unroll
        for (int i = 0; i < DL; ++i) {
            const int64_t at = base + tok * D + sub + kLanesPerRow * i;
            kr[i] = key_ok ? to_float(k[at]) : 0.f;
            vr[i] = key_ok ? to_float(v[at]) : 0.f;
            adk[i] = 0.f;
            adv[i] = 0.f;
        }
        for (int e = list_begin; e < list_end; ++e) {
            const int64_t row0 = (int64_t)row_idx[e] * b;
            for (int c0 = 0; c0 < b; c0 += kChunk) {
                const int nr = min(kChunk, b - c0);
                __syncthreads();
                for (int idx = threadIdx.x; idx < nr * D; idx += kThreads) {
                    const int rr = idx / D, d = idx % D;
                    sq[rr][d] = to_float(q[base + (row0 + c0 + rr) * D + d]);
                    sdo[rr][d] = to_float(dout[base + (row0 + c0 + rr) * D + d]);
                }
                if (threadIdx.x < nr) {
                    const int64_t rt = row0 + c0 + threadIdx.x;
                    float dl = 0.f;
                    for (int d = 0; d < D; ++d) dl = fmaf(to_float(dout[base + rt * D + d]), to_float(out[base + rt * D + d]), dl);
                    const float ls = lse[(int64_t)bh * N + rt];
                    sdelta[threadIdx.x] = dl;
                    slse[threadIdx.x] = ls;
                    slive[threadIdx.x] = (uint8_t)((mask ? mask[rt] != 0 : true) && ls > -CUDART_INF_F);
                }
                __syncthreads();
                for (int rr = 0; rr < nr; ++rr) {
                    float s = 0.f, dp = 0.f;
#pragma unroll
                    for (int i = 0; i < DL; ++i) {
                        s = fmaf(kr[i], sq[rr][sub + kLanesPerRow * i], s);
                        dp = fmaf(vr[i], sdo[rr][sub + kLanesPerRow * i], dp);
                    }
                    s = quad_sum(s);
                    dp = quad_sum(dp);
                    const float p = (key_live && slive[rr]) ? expf(s * scale - slse[rr]) : 0.f;
                    const float ds = p * (dp - sdelta[rr]);
#pragma unroll
                    for (int i = 0; i < DL; ++i) {
                        adv[i] = fmaf(p, sdo[rr][sub + kLanesPerRow * i], adv[i]);
                        adk[i] = fmaf(ds, sq[rr][sub + kLanesPerRow * i], adk[i]);
                    }
                }
            }
        }
        if (key_ok) {
#pragma unroll
            for (int i = 0; i < DL; ++i) {
                store_val(&dk[base + tok * D + sub + kLanesPerRow * i], adk[i] * scale);
                store_val(&dv[base + tok * D + sub + kLanesPerRow * i], adv[i]);
            }
        }
    }
}

template <typename T>
cudaError_t launch_t(const BwdArgs& a, const DeviceLayout& dl) {
    dim3 grid((unsigned)a.nb, (unsigned)(a.B * a.H));
    dim3 block(kThreads);
#define BB_LAUNCH(DD)                                                                                                     \
    attn_bwd_dq_kernel<T, DD><<<grid, block, 0, a.stream>>>((const T*)a.q, (const T*)a.k, (const T*)a.v, (const T*)a.out, a.lse, \
        (const T*)a.dout, dl.row_ptr, dl.col_idx, a.kpm, (T*)a.dq, a.H, a.N, a.b, a.nb, a.scale);                          \
    attn_bwd_dkv_kernel<T, DD><<<grid, block, 0, a.stream>>>((const T*)a.q, (const T*)a.k, (const T*)a.v, (const T*)a.out, a.lse, \
        (const T*)a.dout, dl.col_ptr, dl.row_idx, a.kpm, (T*)a.dk, (T*)a.dv, a.H, a.N, a.b, a.nb, a.scale)
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

cudaError_t launch_attn_bwd_simt(const BwdArgs& a, const DeviceLayout& dl, int* launches) {
    if ((int64_t)a.B * a.H > 65535) return cudaErrorInvalidValue;
    cudaError_t e = a.dtype == BIGBIRD_BF16 ? launch_t<__nv_bfloat16>(a, dl) : launch_t<float>(a, dl);
    if (e == cudaSuccess) *launches += 2;
    return e;
}

}  // namespace bigbird
