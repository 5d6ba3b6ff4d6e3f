// Internal launch interfaces between the C-ABI layer and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "layout.h"

namespace bigbird {

struct FwdArgs {
    const void* q;
    const void* k;
    const void* v;
    const uint8_t* kpm;      // [B, N] or nullptr
    void* out;
    float* lse;              // may be nullptr
    int B, H, D, b, nb;
    int64_t N;
    float scale;
    int dtype;               // BIGBIRD_FP32 / BIGBIRD_BF16
    cudaStream_t stream;
};

struct BwdArgs {
    const void* q;
    const void* k;
    const void* v;
    const void* out;         // the forward result
    const float* lse;        // [B, H, N] from the forward pass
    const void* dout;        // gradient of the loss with respect to out
    const uint8_t* kpm;      // [B, N] or nullptr
    void* dq;
    void* dk;
    void* dv;
    int B, H, D, b, nb;
    int64_t N;
    float scale;
    int dtype;
    cudaStream_t stream;
};

// Per-device scratch owned by the library.
struct DeviceScratch {
    int* status = nullptr;          // [2]: code, detail
    int* counters = nullptr;        // [kCounterSlots * 2] work counters of the dynamic scheduler
    unsigned next_slot = 0;
    unsigned long long* kbits = nullptr;   // [B * nb] one bit per key of a 64-token block (1 = valid)
    size_t kbits_cap = 0;
    float* partials = nullptr;      // partial (O, m, l) of split tiles
    size_t partials_cap = 0;
};
constexpr int kCounterSlots = 64;

// CUDA-core kernel (fp32 arithmetic).  Returns a cudaError_t.  *launches is incremented per kernel enqueued.
cudaError_t launch_attn_fwd_simt(const FwdArgs& a, const DeviceLayout& dl, int* launches);

// CUDA-core gradient kernels (fp32 arithmetic): dq by query block, dk and dv by key block over the transposed lists.
cudaError_t launch_attn_bwd_simt(const BwdArgs& a, const DeviceLayout& dl, int* launches);

// tcgen05 kernel (bf16 operands).  Returns a BIGBIRD_* code; *cuda_err receives the cudaError_t on BIGBIRD_ECUDA.
int launch_attn_fwd_sm100(const FwdArgs& a, const bigbird_layout& L, const DeviceLayout& dl, DeviceScratch& sc,
                          int* launches, cudaError_t* cuda_err);

// One-thread kernel whose bounded wait is left to expire (about two seconds); sets the device status word.
cudaError_t launch_wait_expiry_selftest(DeviceScratch& sc, cudaStream_t stream);

}  // namespace bigbird
