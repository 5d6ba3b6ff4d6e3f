// CUDA-core BigBird attention forward (arXiv 2007.14062, Eq. (AT) over the block lists of App. D).
// fp32 arithmetic throughout; the path for fp32 tensors and an independent check for the tensor-core kernel.
//
// One CTA per (batch*head, query block, group of 8 query rows).  A warp shares a query row: for the scores each lane
// takes a thirty-second of a chunk's keys (and the whole dot product of each), for the output a thirty-second of the head
// dimension.  Key blocks are staged through shared memory (64 keys at a time for D <= 64, 32 for D = 128) and folded
// into a running (max, sum, output) triple per row (online softmax).  The next chunk's K and V are already on their
// way into registers while the current one is being used.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "kernels.h"
#include "../../include/bigbird.h"

namespace bigbird {
namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerRow = 32;
constexpr int kRowsPerCta = kThreads / kLanesPerRow;

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
    constexpr int DL = D / kLanesPerRow;           // head dims per lane for the output: d = DL*sub .. DL*sub + DL - 1
    constexpr int KC = D <= 64 ? 64 : 32;          // keys per staged chunk
    constexpr int PF = KC * D / kThreads;          // elements of K (and of V) each thread moves per chunk
    // rows padded by four floats: 16-byte aligned for vector loads, and the keys a warp reads at once fall
    // into different banks
    __shared__ __align__(16) float sk[KC][D + 4];
    __shared__ __align__(16) float sv[KC][D + 4];
    __shared__ uint8_t svalid[KC];

    const int groups = (b + kRowsPerCta - 1) / kRowsPerCta;
    const int j = blockIdx.x / groups;
    const int row = (blockIdx.x % groups) * kRowsPerCta + threadIdx.x / kLanesPerRow;
    const int bh = blockIdx.y;
    const int h = bh % H, batch = bh / H;
    const int sub = threadIdx.x % kLanesPerRow;
    const int64_t base = (int64_t)bh * N * D;
    const int list_begin = row_ptr[(int64_t)h * nb + j], list_end = row_ptr[(int64_t)h * nb + j + 1];
    const uint8_t* mask = kpm ? kpm + (int64_t)batch * N : nullptr;
    const bool row_ok = row < b;
    const int64_t tok = (int64_t)j * b + row;

    // Scores: lane t of a row takes the keys t, t + 32, ... of a chunk and the whole dot product of each (no
    // exchange between lanes per key).  Output: lane t accumulates the head dims DL t .. DL t + DL - 1 over every key of
    // the chunk; the probabilities pass from the first layout to the second through shared memory.
    constexpr int KL = KC / kLanesPerRow;           // keys per lane per chunk
    __shared__ float sp[kRowsPerCta][KC];
    const int rloc = threadIdx.x / kLanesPerRow;
    float qr[D], o[DL];
#pragma unroll
    for (int d = 0; d < D; ++d) qr[d] = row_ok ? to_float(q[base + tok * D + d]) * scale : 0.f;
#pragma unroll
    for (int i = 0; i < DL; ++i) o[i] = 0.f;
    float m = -CUDART_INF_F, l = 0.f;               // l: this lane's keys only, summed over the lanes at the end

    // chunks of the key sweep: (list entry, offset inside the key block)
    const int chunks_per_block = (b + KC - 1) / KC;
    const int n_chunks = (list_end - list_begin) * chunks_per_block;
    float pk[PF], pv[PF];
    uint8_t pm = 1;
    auto fetch = [&](int ci) {                      // chunk ci from global memory into registers
        const int64_t key0 = (int64_t)col_idx[list_begin + ci / chunks_per_block] * b + (ci % chunks_per_block) * KC;
        const int nk = min(KC, b - (ci % chunks_per_block) * KC);
#pragma unroll
        for (int t = 0; t < PF; ++t) {
            const int idx = threadIdx.x + t * kThreads, kk = idx / D, d = idx % D;
            const bool in = kk < nk;
            pk[t] = in ? to_float(k[base + (key0 + kk) * D + d]) : 0.f;
            pv[t] = in ? to_float(v[base + (key0 + kk) * D + d]) : 0.f;
        }
        if (threadIdx.x < KC) pm = (threadIdx.x < nk && (mask ? mask[key0 + threadIdx.x] != 0 : true)) ? 1 : 0;
    };
    if (n_chunks > 0) fetch(0);
    for (int ci = 0; ci < n_chunks; ++ci) {
        __syncthreads();                            // the previous chunk has been used
#pragma unroll
        for (int t = 0; t < PF; ++t) {
            const int idx = threadIdx.x + t * kThreads, kk = idx / D, d = idx % D;
            sk[kk][d] = pk[t];
            sv[kk][d] = pv[t];
        }
        if (threadIdx.x < KC) svalid[threadIdx.x] = pm;
        __syncthreads();
        if (ci + 1 < n_chunks) fetch(ci + 1);       // in flight while this chunk is being used
        float s[KL];
        float cmax = -CUDART_INF_F;
#pragma unroll
        for (int u = 0; u < KL; ++u) {
            const int kk = sub + kLanesPerRow * u;
            float acc = 0.f;
#pragma unroll
            for (int d = 0; d < D; d += 4) {
                const float4 k4 = *reinterpret_cast<const float4*>(&sk[kk][d]);
                acc = fmaf(qr[d], k4.x, acc);
                acc = fmaf(qr[d + 1], k4.y, acc);
                acc = fmaf(qr[d + 2], k4.z, acc);
                acc = fmaf(qr[d + 3], k4.w, acc);
            }
            s[u] = svalid[kk] ? acc : -CUDART_INF_F;         // keys beyond the block's end were staged as invalid
            cmax = fmaxf(cmax, s[u]);
        }
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 1));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 2));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 4));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
        if (cmax == -CUDART_INF_F) continue;        // whole chunk masked (uniform across the CTA: the mask is per key)
        const float m_new = fmaxf(m, cmax);
        const float alpha = expf(m - m_new);        // m = -inf on the first chunk gives 0
        l *= alpha;
#pragma unroll
        for (int i = 0; i < DL; ++i) o[i] *= alpha;
#pragma unroll
        for (int u = 0; u < KL; ++u) {
            const float p = expf(s[u] - m_new);     // exp(-inf) = 0 for masked keys
            l += p;
            sp[rloc][sub + kLanesPerRow * u] = p;
        }
        __syncwarp();                               // a row is one warp
#pragma unroll
        for (int kk = 0; kk < KC; ++kk) {
            const float p = sp[rloc][kk];
            if constexpr (DL >= 2) {
#pragma unroll
                for (int i = 0; i < DL; i += 2) {
                    const float2 v2 = *reinterpret_cast<const float2*>(&sv[kk][DL * sub + i]);
                    o[i] = fmaf(p, v2.x, o[i]);
                    o[i + 1] = fmaf(p, v2.y, o[i + 1]);
                }
            } else {
                o[0] = fmaf(p, sv[kk][sub], o[0]);
            }
        }
        __syncwarp();
        m = m_new;
    }
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    l += __shfl_xor_sync(0xffffffffu, l, 4);
    l += __shfl_xor_sync(0xffffffffu, l, 8);
    l += __shfl_xor_sync(0xffffffffu, l, 16);
    if (row_ok) {
        const bool q_valid = mask ? mask[tok] != 0 : true;
        const bool any = q_valid && l > 0.f;
        const float inv = any ? 1.f / l : 0.f;
#pragma unroll
        for (int i = 0; i < DL; ++i) store_val(&out[base + tok * D + DL * sub + i], o[i] * inv);
        if (lse && sub == 0) lse[(int64_t)bh * N + tok] = any ? m + logf(l) : -CUDART_INF_F;
    }
}

template <typename T>
cudaError_t launch_t(const FwdArgs& a, const DeviceLayout& dl) {
    dim3 grid((unsigned)(a.nb * ((a.b + kRowsPerCta - 1) / kRowsPerCta)), (unsigned)(a.B * a.H));
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
