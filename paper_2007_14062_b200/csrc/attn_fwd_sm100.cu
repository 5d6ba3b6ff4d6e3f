// BigBird block-sparse attention forward on Blackwell tensor cores (sm_100a).
//
// What is computed: Eq. (AT) of arXiv 2007.14062 (softmax attention restricted to the out-neighbours of each
// query) over the block graph of App. D.  How, on B200:
//
//   * Two query blocks are stacked into one 128-row tile so that every tcgen05.mma runs at M = 128.  The tile
//     walks a list of key blocks prepared on the host; each is attended by both halves of the tile or by one.
//     The MMAs always cover all 128 rows; rows that do not attend a key block get probability zero for it.
//   * A producer thread fetches Q once per tile and the K and V blocks with TMA (128-byte swizzle) straight
//     from the [B, H, N, D] tensors into a shared-memory ring: nothing is gathered or packed in HBM.
//   * Key blocks are processed two at a time (one "step").  Their K tiles land in adjacent ring slots, so that
//     S = Q K^T of a step is one N = 128 tcgen05.mma per 16 head dimensions (an MMA instruction costs its issuing
//     thread about the same time whatever its N, so wide MMAs are the cheap ones).  O += P V follows with P read
//     from tensor memory.
//   * Four softmax warps, one thread per row of the tile: the thread pulls its (up to) 128 scores into registers
//     with tcgen05.ld and hands the score columns back at once, so that the next step's Q K^T runs under this
//     step's exponentials; it applies the key-padding mask, takes the row maximum, exponentiates (base 2, fp32),
//     sums, and writes bf16 probabilities with tcgen05.st (zeros for key blocks its half of the tile does not
//     attend); the previous step's P V runs under the first half of that.  The accumulator is rescaled only
//     when the running maximum grows by more than 2^8.  The output of a tile is written during the first step
//     of the next tile.
//   * A global-row tile of a long sequence is cut along the keys into parts that are separate work items; each
//     writes its unnormalised accumulator and (max, sum) per row to scratch, and a small merge kernel combines
//     the parts in a fixed order.
//   * CTAs are persistent and draw work from a global counter: global-row tiles first, then the sparse tiles
//     in (batch, head)-major order.  Two CTAs share an SM so that one's softmax overlaps the other's MMAs.
//
// Every wait on an mbarrier is bounded: on expiry the kernel records BIGBIRD_ETIMEOUT and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>
#include <vector>

#include "kernels.h"
#include "../../include/bigbird.h"

namespace bigbird {
namespace {

// ------------------------------------------------------------------------------------------------ constants
constexpr int kBlock = 64;                 // tokens per block (b) and head dimension (D)
constexpr int kTileBytes = kBlock * kBlock * 2;      // one 64x64 bf16 tile
constexpr int kStepChunks = 2;             // key blocks per step
constexpr int kRingGroups = 4;             // ring of groups of kStepChunks adjacent tiles (the K or the V blocks of one step)
constexpr int kGroupBytes = kStepChunks * kTileBytes;
constexpr int kThreads = 256;              // warp 0 TMA, warp 1 MMA issuer, warp 2 scheduler, warp 3 idle, warps 4..7 softmax
constexpr int kSoftmaxWarps = 4;
#ifndef BB_REGS_LIGHT
#define BB_REGS_LIGHT 72
#define BB_REGS_SOFTMAX 184
#endif
constexpr int kRegsLight = BB_REGS_LIGHT;             // registers per thread of warps 0..3 after setmaxnreg
constexpr int kRegsSoftmax = BB_REGS_SOFTMAX;          // registers per thread of warps 4..7 after setmaxnreg
constexpr int kTmemCols = 256;
constexpr int kColS = 0;                   // scores: kStepChunks x 64 fp32 columns
constexpr int kColP = kStepChunks * 64;    // probabilities: kStepChunks x 32 columns of packed bf16 pairs
constexpr int kColO = kColP + kStepChunks * 32;   // output accumulator: 64 fp32 columns
constexpr float kRescaleThreshold = 8.0f;  // in log2 units
constexpr long long kWaitLimitCycles = 4000000000ll;   // about two seconds
constexpr int kSchedSlots = 3;
constexpr int kPartialFloats = 128 * 64 + 2 * 128;   // one part of a split tile: O[128][64], max[128], sum[128]
constexpr int kSegChunks = 96;             // live key blocks per posted segment of a tile (a multiple of kStepChunks)
static_assert(kColO + 64 <= kTmemCols && kSegChunks % kStepChunks == 0, "tensor-memory and segment layout");

// A key block of a tile after the key-padding mask has been applied.
struct __align__(16) ChunkEntry {
    int c;                         // key block
    int who;                       // bits 0..1: kBothHalves, kUpperHalf or kLowerHalf (the halves of the tile that attend it);
                                   // bit 2 (kHasPadding): some of its keys are padding
    unsigned long long kb;         // valid-key bits (never 0: blocks that are entirely padding are dropped)
};
enum { kSegFirst = 1, kSegLast = 2, kSegLive = 4 };
enum { kWhoMask = 3, kHasPadding = 4, kNoChunk = 3 };
struct __align__(16) WorkSlot {
    int w;                         // work index, -1 = no more work
    int bh, batch, qa, qb;
    int n_chunks;
    int flags;
    int part_slot;                 // >= 0: the tile is one part of a split tile and writes partial results there
    unsigned long long qbits_a, qbits_b;
    ChunkEntry chunks[kSegChunks];         // step s of the segment covers chunks [kStepChunks s, kStepChunks (s + 1))
};

struct __align__(16) SmemCtl {
    unsigned long long full[kRingGroups];
    unsigned long long empty[kRingGroups];
    unsigned long long q_full[2], q_empty[2];
    unsigned long long s_full, s_free, p_full, pv_done;
    unsigned long long sched_full[kSchedSlots], sched_empty[kSchedSlots];
    unsigned tmem_base;
    int abort_flag;
    WorkSlot slot[kSchedSlots];
};
constexpr int kSmemQ = 0;
constexpr int kSmemRing = 4 * kTileBytes;              // two Q buffers of two tiles each come first
constexpr int kSmemCtl = kSmemRing + kRingGroups * kGroupBytes;
constexpr int kSmemBytes = kSmemCtl + (int)sizeof(SmemCtl) + 1024;   // + slack for the 1024-byte alignment

struct KernelParams {
    __nv_bfloat16* out;
    float* lse;
    const unsigned long long* kbits;   // [B * nb] or nullptr
    const Item* items;
    const Step* steps;
    int* counter;                      // [2]: next work index, finished CTAs
    int* status;                       // [2]: code, detail
    int items_per_head, heavy_per_head;
    int BH, H, nb;
    int total_work;
    float scale_log2;
    float* partials;                   // [BH * split_tiles_per_head * max_parts][kPartialFloats] or nullptr
    int split_tiles_per_head, max_parts;
};

// ------------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if the wait expired or another thread of the CTA already gave up.  The limit is
// counted in SM clock cycles (a read of the cycle counter is cheap, unlike one of the global nanosecond timer)
// and the counter is first read only after 64 failed tries.
__device__ __forceinline__ bool mbar_wait_slow(unsigned long long* bar, unsigned parity, SmemCtl* ctl, int* status, int code) {
    long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*(volatile int*)&ctl->abort_flag) return false;
            const long long now = clock64();
            if (it == 63u) t0 = now;
            if (now - t0 > kWaitLimitCycles) {
                if (atomicCAS(status, 0, BIGBIRD_ETIMEOUT) == 0) status[1] = code;
                *(volatile int*)&ctl->abort_flag = 1;
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, SmemCtl* ctl, int* status, int code) {
    if (__builtin_expect(mbar_try(bar, parity), 1)) return true;
    return mbar_wait_slow(bar, parity, ctl, status, code);
}

__device__ __forceinline__ void tma_load_tile(void* dst, const CUtensorMap* tm, int row, unsigned long long* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"((unsigned long long)tm), "r"(0), "r"(row), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc, unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(unsigned d_tmem, unsigned a_tmem, unsigned long long b_desc, unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart (a dense 64-wide bf16 tile).
__device__ __forceinline__ unsigned long long smem_desc_sw128(unsigned addr) {
    return (unsigned long long)((addr & 0x3FFFFu) >> 4)
         | (1ull << 16)                       // leading byte offset (unused for a single 128-byte atom)
         | ((unsigned long long)(1024 >> 4) << 32)   // stride byte offset: next group of 8 rows
         | (1ull << 46)                       // descriptor version of sm_100
         | (2ull << 61);                      // SWIZZLE_128B
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 64 (Q K^T adds 64 per further key block); B is K-major (K^T) or MN-major (V).
constexpr unsigned kIdescQK64 = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);   // N field (bits 17..22) = N / 8
constexpr unsigned kIdescPV = kIdescQK64 | (1u << 16);

#define BB_REP32(F, o) F(o+0), F(o+1), F(o+2), F(o+3), F(o+4), F(o+5), F(o+6), F(o+7), F(o+8), F(o+9), F(o+10), F(o+11), \
    F(o+12), F(o+13), F(o+14), F(o+15), F(o+16), F(o+17), F(o+18), F(o+19), F(o+20), F(o+21), F(o+22), F(o+23), \
    F(o+24), F(o+25), F(o+26), F(o+27), F(o+28), F(o+29), F(o+30), F(o+31)
#define BB_OUT(i) "=r"(u[i])
#define BB_IN(i) "r"(u[i])
__device__ __forceinline__ void tmem_ld64(unsigned taddr, float* r) {
    unsigned* u = reinterpret_cast<unsigned*>(r);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
        "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
        "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : BB_REP32(BB_OUT, 0), BB_REP32(BB_OUT, 32) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, float* r) {
    unsigned* u = reinterpret_cast<unsigned*>(r);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : BB_REP32(BB_OUT, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(unsigned taddr, const unsigned* u) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::BB_REP32(BB_IN, 0), "r"(taddr) : "memory");
}
#define BB_REP16(F, o) F(o+0), F(o+1), F(o+2), F(o+3), F(o+4), F(o+5), F(o+6), F(o+7), F(o+8), F(o+9), F(o+10), F(o+11), \
    F(o+12), F(o+13), F(o+14), F(o+15)
__device__ __forceinline__ void tmem_ld16(unsigned taddr, float* r) {
    unsigned* u = reinterpret_cast<unsigned*>(r);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : BB_REP16(BB_OUT, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(unsigned taddr, const unsigned* u) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::BB_REP16(BB_IN, 0), "r"(taddr) : "memory");
}
#undef BB_OUT
#undef BB_IN
__device__ __forceinline__ void tmem_st32_zero(unsigned taddr) {
    const unsigned z = 0;
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%1], "
        "{%0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, "
        "%0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0};"
        ::"r"(z), "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16_zero(unsigned taddr) {
    const unsigned z = 0;
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%1], "
        "{%0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0, %0};"
        ::"r"(z), "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// (x0, x1) * a + b on the packed fp32 pipe
__device__ __forceinline__ void ffma2(float& r0, float& r1, float x0, float x1, float a, float b) {
    asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %4}; mov.b64 rc, {%5, %5}; "
        "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0, %1}, rd; }"
        : "=f"(r0), "=f"(r1) : "f"(x0), "f"(x1), "f"(a), "f"(b));
}
__device__ __forceinline__ void fadd2(float& r0, float& r1, float x0, float x1) {
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%0, %1}; mov.b64 rb, {%2, %3}; add.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "+f"(r0), "+f"(r1) : "f"(x0), "f"(x1));
}
__device__ __forceinline__ void fmul2(float& r0, float& r1, float a) {
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%0, %1}; mov.b64 rb, {%2, %2}; mul.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "+f"(r0), "+f"(r1) : "f"(a));
}

// ------------------------------------------------------------------------------------------------ schedule helpers
__device__ __forceinline__ unsigned long long key_bits(const KernelParams& p, int batch, int c) {
    if (c < 0) return 0ull;
    return p.kbits ? p.kbits[(size_t)batch * p.nb + c] : ~0ull;
}
__device__ __forceinline__ float row_max64(const float* s) {
    float mx0 = max3(s[0], s[1], s[2]), mx1 = max3(s[3], s[4], s[5]), mx2 = max3(s[6], s[7], s[8]), mx3 = max3(s[9], s[10], s[11]);
#pragma unroll
    for (int j = 12; j < 60; j += 8) {
        mx0 = max3(mx0, s[j], s[j + 1]);
        mx1 = max3(mx1, s[j + 2], s[j + 3]);
        mx2 = max3(mx2, s[j + 4], s[j + 5]);
        mx3 = max3(mx3, s[j + 6], s[j + 7]);
    }
    return fmaxf(max3(mx0, mx1, fmaxf(s[60], s[61])), max3(mx2, mx3, fmaxf(s[62], s[63])));
}

// ------------------------------------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(kThreads, 2)
attn_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const KernelParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + kSmemCtl);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kRingGroups; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->q_full[i], 1); mbar_init(&ctl->q_empty[i], 1); }
        mbar_init(&ctl->s_full, 1);
        mbar_init(&ctl->s_free, kSoftmaxWarps * 32);    // every softmax thread arrives itself: cheaper than
        mbar_init(&ctl->p_full, kSoftmaxWarps * 32);    // converging the warp and electing a lane
        mbar_init(&ctl->pv_done, 1);
        for (int i = 0; i < kSchedSlots; ++i) { mbar_init(&ctl->sched_full[i], 1); mbar_init(&ctl->sched_empty[i], 2 + kSoftmaxWarps * 32); }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = *(volatile unsigned*)&ctl->tmem_base;

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLight));
        if (warp == 2) {
            // ================================================================= scheduler: fetch work, post live key blocks
            unsigned sched_n = 0;
            bool ok = true;
            const unsigned lt_mask = (1u << lane) - 1u;
            while (ok) {
                int w = 0;
                if (lane == 0) w = atomicAdd(&p.counter[0], 1);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (w >= p.total_work) w = -1;
                // decode the work index: global-row tiles of every (batch, head) first, then the sparse tiles
                int bh = 0, it = 0;
                Item item{};
                if (w >= 0) {
                    const int heavy_total = p.BH * p.heavy_per_head;
                    if (w < heavy_total) {
                        bh = w / p.heavy_per_head;
                        it = w - bh * p.heavy_per_head;
                    } else {
                        const int sparse = p.items_per_head - p.heavy_per_head;
                        const int w2 = w - heavy_total;
                        bh = w2 / sparse;
                        it = p.heavy_per_head + (w2 - bh * sparse);
                    }
                    item = p.items[(size_t)(bh % p.H) * p.items_per_head + it];
                }
                const int batch = bh / p.H;
                const unsigned long long qbits_a = w >= 0 ? key_bits(p, batch, item.qa) : 0ull;
                const unsigned long long qbits_b = w >= 0 ? key_bits(p, batch, item.qb) : 0ull;
                const bool tile_live = (qbits_a | qbits_b) != 0ull;      // a tile whose query rows are all padding is skipped
                const int n_raw = (w >= 0 && tile_live) ? item.step_count : 0;
                int i0 = 0;
                bool first = true;
                do {
                    const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
                    ok = mbar_wait(&ctl->sched_empty[ss], sp ^ 1u, ctl, p.status, 11);
                    if (!ok) break;
                    WorkSlot* slot = &ctl->slot[ss];
                    int count = 0;
                    while (i0 < n_raw && count <= kSegChunks - 32) {
                        const int i = i0 + lane;
                        ChunkEntry e{-1, 0, 0ull};
                        bool alive = false;
                        if (i < n_raw) {
                            const Step s = p.steps[item.step_begin + i];
                            // halves whose query rows are all padding do not attend anything
                            const bool ua = s.who != kLowerHalf && qbits_a != 0ull;
                            const bool ub = s.who != kUpperHalf && qbits_b != 0ull;
                            e.c = s.c;
                            e.kb = key_bits(p, batch, s.c);
                            e.who = ((ua && ub) ? kBothHalves : (ua ? kUpperHalf : kLowerHalf)) | (e.kb != ~0ull ? kHasPadding : 0);
                            alive = e.kb != 0ull && (ua || ub);
                        }
                        const unsigned bal = __ballot_sync(0xffffffffu, alive);
                        if (alive) slot->chunks[count + __popc(bal & lt_mask)] = e;
                        count += __popc(bal);
                        i0 += 32;
                    }
                    if (lane == 0) {
                        slot->w = w;
                        slot->bh = bh;
                        slot->batch = batch;
                        slot->qa = item.qa;
                        slot->qb = item.qb;
                        slot->n_chunks = count;
                        slot->flags = (first ? kSegFirst : 0) | (i0 >= n_raw ? kSegLast : 0) | (tile_live ? kSegLive : 0);
                        slot->qbits_a = qbits_a;
                        slot->qbits_b = qbits_b;
                        slot->part_slot = (w >= 0 && item.nparts > 1) ? ((bh * p.split_tiles_per_head + item.tile) * p.max_parts + item.part) : -1;
                    }
                    __threadfence_block();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->sched_full[ss]);
                    ++sched_n;
                    first = false;
                } while (i0 < n_raw);
                if (w < 0) break;
            }
        } else if (warp == 0 && lane == 0) {
            // ================================================================= TMA producer
            // Ring order = the order in which the MMA thread consumes groups: K of step i, then V of step i-1.
            unsigned ring_n = 0, q_n = 0, sched_n = 0;
            bool ok = true;
            // the (up to two) blocks c[0..cnt) of K or V into the next group of adjacent ring slots
            auto load_group = [&](const CUtensorMap* tm, int bh, const int* c, int cnt) -> bool {
                const unsigned g = ring_n % kRingGroups, ph = (ring_n / kRingGroups) & 1u;
                if (!mbar_wait(&ctl->empty[g], ph ^ 1u, ctl, p.status, 10)) return false;
                mbar_expect_tx(&ctl->full[g], cnt * kTileBytes);
#pragma unroll
                for (int j = 0; j < kStepChunks; ++j)
                    if (j < cnt) tma_load_tile(smem + kSmemRing + g * kGroupBytes + j * kTileBytes, tm, (bh * p.nb + c[j]) * kBlock, &ctl->full[g]);
                ++ring_n;
                return true;
            };
            int pend_n = 0, pend_bh = 0, pend_c[kStepChunks] = {0, 0};
            while (ok) {
                const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
                if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 13)) break;
                const WorkSlot* slot = &ctl->slot[ss];
                const int w = slot->w, flags = slot->flags, bh = slot->bh, n = slot->n_chunks;
                if (w >= 0 && (flags & kSegLive)) {
                    if (flags & kSegFirst) {
                        const int qa = slot->qa, qb = slot->qb;
                        const unsigned qs = q_n & 1u;
                        ok = mbar_wait(&ctl->q_empty[qs], ((q_n >> 1) & 1u) ^ 1u, ctl, p.status, 12);
                        if (!ok) break;
                        mbar_expect_tx(&ctl->q_full[qs], qb >= 0 ? 2 * kTileBytes : kTileBytes);
                        tma_load_tile(smem + kSmemQ + qs * 2 * kTileBytes, &tm_q, (bh * p.nb + qa) * kBlock, &ctl->q_full[qs]);
                        if (qb >= 0) tma_load_tile(smem + kSmemQ + qs * 2 * kTileBytes + kTileBytes, &tm_q, (bh * p.nb + qb) * kBlock, &ctl->q_full[qs]);
                        ++q_n;
                    }
                    for (int i = 0; i < n && ok; i += kStepChunks) {
                        int c[kStepChunks];
                        const int cnt = min(kStepChunks, n - i);
#pragma unroll
                        for (int j = 0; j < kStepChunks; ++j) c[j] = j < cnt ? slot->chunks[i + j].c : 0;
                        ok = load_group(&tm_k, bh, c, cnt);
                        if (ok && pend_n > 0) ok = load_group(&tm_v, pend_bh, pend_c, pend_n);
#pragma unroll
                        for (int j = 0; j < kStepChunks; ++j) pend_c[j] = c[j];
                        pend_n = cnt;
                        pend_bh = bh;
                    }
                }
                mbar_arrive(&ctl->sched_empty[ss]);
                ++sched_n;
                if (w < 0) {
                    if (ok && pend_n > 0) load_group(&tm_v, pend_bh, pend_c, pend_n);
                    break;
                }
            }
        } else if (warp == 1 && lane == 0) {
            // ================================================================= MMA issuer
            unsigned ring_n = 0, q_n = 0, sched_n = 0, grp_n = 0, pv_n = 0;   // grp_n: steps whose Q K^T was issued
            bool ok = true;
            auto qk = [&](int cnt, unsigned qs) -> bool {   // S[:, 0 .. 64 cnt) = Q K^T with the K blocks of the next ring group
                const unsigned g = ring_n % kRingGroups, ph = (ring_n / kRingGroups) & 1u;
                if (!mbar_wait(&ctl->full[g], ph, ctl, p.status, 20)) return false;
                tc_fence_after();
                // the blocks of a group are adjacent: their 64 cnt rows form one K-major operand
                const unsigned long long q_desc = smem_desc_sw128(smem_u32(smem + kSmemQ + qs * 2 * kTileBytes));
                const unsigned long long k_desc = smem_desc_sw128(smem_u32(smem + kSmemRing + g * kGroupBytes));
                const unsigned idesc = kIdescQK64 + ((unsigned)(cnt - 1) << 20);           // N = 64 cnt
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)          // 16 head dims (32 bytes inside the swizzled row) per MMA
                    mma_ss(tmem + kColS, q_desc + (unsigned long long)(kk * 2), k_desc + (unsigned long long)(kk * 2), idesc, kk > 0);
                tc_commit(&ctl->empty[g]);
                ++ring_n;
                return true;
            };
            bool pend_fresh = false;                    // the pending P V is the first of its tile: it overwrites O
            bool tile_fresh = false, q_unseen = false;
            int pend_n = 0;
            auto pending_pv = [&]() -> bool {           // O (+)= sum_j P_j V_j with the V blocks of the next ring group
                if (pend_n == 0) return true;
                if (!mbar_wait(&ctl->p_full, pv_n & 1u, ctl, p.status, 22)) return false;
                const unsigned g = ring_n % kRingGroups, ph = (ring_n / kRingGroups) & 1u;
                if (!mbar_wait(&ctl->full[g], ph, ctl, p.status, 21)) return false;
                tc_fence_after();
                const unsigned long long v_desc = smem_desc_sw128(smem_u32(smem + kSmemRing + g * kGroupBytes));
#pragma unroll
                for (int j = 0; j < kStepChunks; ++j) {
                    if (j < pend_n) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)  // 16 keys per MMA: 8 packed columns of P_j, two 8-row groups of V_j
                            mma_ts(tmem + kColO, tmem + kColP + 32 * j + kk * 8, v_desc + (unsigned long long)((j * kTileBytes + kk * 2048) >> 4), kIdescPV,
                                   (j > 0 || kk > 0 || !pend_fresh) ? 1u : 0u);
                    }
                }
                tc_commit(&ctl->empty[g]);
                tc_commit(&ctl->pv_done);
                ++ring_n;
                ++pv_n;
                pend_n = 0;
                pend_fresh = false;
                return true;
            };
            while (ok) {
                const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
                if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 23)) break;
                const WorkSlot* slot = &ctl->slot[ss];
                const int w = slot->w, flags = slot->flags, n = slot->n_chunks;
                if (w >= 0 && (flags & kSegLive)) {
                    if (flags & kSegFirst) {
                        ++q_n;                          // this tile's Q sits in buffer (q_n - 1) & 1
                        q_unseen = true;
                        tile_fresh = true;
                    }
                    const unsigned qs = (q_n - 1) & 1u, qph = ((q_n - 1) >> 1) & 1u;
                    for (int i = 0; i < n && ok; i += kStepChunks) {
                        // the softmax threads must have pulled the previous scores out of tensor memory
                        if (grp_n > 0) {
                            ok = mbar_wait(&ctl->s_free, (grp_n - 1) & 1u, ctl, p.status, 25);
                            if (!ok) break;
                        }
                        if (q_unseen) {
                            ok = mbar_wait(&ctl->q_full[qs], qph, ctl, p.status, 24);
                            if (!ok) break;
                            q_unseen = false;
                        }
                        tc_fence_after();
                        const int cnt = min(kStepChunks, n - i);
                        ok = qk(cnt, qs);
                        if (!ok) break;
                        tc_commit(&ctl->s_full);
                        ++grp_n;
                        // the previous step's P V goes behind this step's Q K^T
                        ok = pending_pv();
                        pend_n = cnt;
                        pend_fresh = tile_fresh;
                        tile_fresh = false;
                    }
                    if (!ok) break;
                    if (flags & kSegLast) {
                        if (q_unseen) {                 // a tile without a live key block: its Q still has to land
                            ok = mbar_wait(&ctl->q_full[qs], qph, ctl, p.status, 26);
                            if (!ok) break;
                            q_unseen = false;
                        }
                        tc_commit(&ctl->q_empty[qs]);   // every Q K^T of the tile has been issued
                    }
                }
                mbar_arrive(&ctl->sched_empty[ss]);
                ++sched_n;
                if (w < 0) {
                    pending_pv();
                    break;
                }
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        // ===================================================================== softmax + epilogue (128 threads, one per row)
        const int quad = warp & 3;                      // tensor-memory lanes this warp may touch: 32*quad .. +31
        const int row = quad * 32 + lane;               // row of the 128-row tile
        const bool lower = row >= kBlock;
        const int my_who = lower ? kLowerHalf : kUpperHalf;
        const unsigned lane_addr = tmem + ((unsigned)(quad * 32) << 16);
        const float sl2 = p.scale_log2;
        unsigned sched_n = 0, grp_n = 0;
        bool ok = true;
        float m_ref = -INFINITY, l_sum = 0.f;
        bool o_dirty = false;                           // has any P V been issued for this tile yet
        // output of the previous tile, written once its last P V is known to be complete
        bool pend_out = false, pend_partial = false;
        float pend_inv = 0.f;
        uint4* pend_dst = nullptr;
        auto write_out = [&]() {                        // the 64 accumulator columns of this thread's row
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                float o[32];
                tmem_ld32(lane_addr + kColO + c * 32, o);
                tmem_wait_ld();
                if (pend_partial) {                     // one part of a split tile: the raw fp32 accumulator
                    float4* d4 = reinterpret_cast<float4*>(pend_dst) + 8 * c;
#pragma unroll
                    for (int j = 0; j < 8; ++j) d4[j] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                } else {                                // pend_inv is 0 for rows that must come out as zeros
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v4;
                        v4.x = pack_bf16(o[8 * j + 0] * pend_inv, o[8 * j + 1] * pend_inv);
                        v4.y = pack_bf16(o[8 * j + 2] * pend_inv, o[8 * j + 3] * pend_inv);
                        v4.z = pack_bf16(o[8 * j + 4] * pend_inv, o[8 * j + 5] * pend_inv);
                        v4.w = pack_bf16(o[8 * j + 6] * pend_inv, o[8 * j + 7] * pend_inv);
                        pend_dst[4 * c + j] = v4;
                    }
                }
            }
            pend_out = false;
        };
        // -inf over the scores of padded keys of one key block, in tensor memory (s: 64 scratch registers)
        auto mask_scores = [&](float* s, unsigned taddr, unsigned long long kb) {
            tmem_ld64(taddr, s);
            tmem_wait_ld();
#pragma unroll
            for (int t = 0; t < 64; ++t) s[t] = ((kb >> t) & 1ull) ? s[t] : -INFINITY;
            tmem_st32(taddr, reinterpret_cast<unsigned*>(s));
            tmem_st32(taddr + 32, reinterpret_cast<unsigned*>(s + 32));
            tmem_wait_st();
        };
        // exponentials of the 64 scores of one key block, packed in place: afterwards s[0..31] hold the bit
        // patterns of the 32 words of bf16 probability pairs
        auto exp_pack = [&](float* s, float neg_m, float& sum0, float& sum1) {
#pragma unroll
            for (int t = 0; t < 64; t += 2) {
                float t0, t1;
                ffma2(t0, t1, s[t], s[t + 1], sl2, neg_m);
                const float p0 = ex2(t0), p1 = ex2(t1);
                fadd2(sum0, sum1, p0, p1);
                s[t >> 1] = __uint_as_float(pack_bf16(p0, p1));
            }
        };
        while (ok) {
            const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
            if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 30)) break;
            const WorkSlot* slot = &ctl->slot[ss];
            const int w = slot->w, flags = slot->flags, n = slot->n_chunks;
            if (w < 0) {
                if (pend_out) {                         // warp-uniform; the last P V of all
                    ok = mbar_wait(&ctl->pv_done, (grp_n - 1) & 1u, ctl, p.status, 35);
                    if (!ok) break;
                    tc_fence_after();
                    write_out();
                }
                break;
            }
            const bool live = flags & kSegLive;
            if (flags & kSegFirst) {
                m_ref = -INFINITY;
                l_sum = 0.f;
                o_dirty = false;
            }
            for (int i = 0; i < n && ok; i += kStepChunks) {
                const ChunkEntry* e = &slot->chunks[i];
                const int cnt = min(kStepChunks, n - i);
                // which of the step's key blocks my half of the tile attends (warp-uniform)
                const int who0 = e[0].who, who1 = cnt > 1 ? e[1].who : kNoChunk;
                const bool mine0 = (who0 & kWhoMask) == kBothHalves || (who0 & kWhoMask) == my_who;
                const bool mine1 = (who1 & kWhoMask) == kBothHalves || (who1 & kWhoMask) == my_who;
                ok = mbar_wait(&ctl->s_full, grp_n & 1u, ctl, p.status, 31);
                if (!ok) break;
                tc_fence_after();
                float s[128];
                // A key block with padded keys (rare: the one holding a sequence's end) gets -inf written over their
                // scores in tensor memory first, so that the common path below carries no masking code at all.
                if (__builtin_expect(((who0 | who1) & kHasPadding) != 0, 0)) {
                    if (mine0 && (who0 & kHasPadding)) mask_scores(s, lane_addr + kColS, e[0].kb);
                    if (mine1 && (who1 & kHasPadding)) mask_scores(s, lane_addr + kColS + 64, e[1].kb);
                }
                if (mine0) tmem_ld64(lane_addr + kColS, s);
                if (mine1) tmem_ld64(lane_addr + kColS + 64, s + 64);
                tmem_wait_ld();
                // the score columns are free again: the next step's Q K^T may overwrite them
                tc_fence_before();
                mbar_arrive(&ctl->s_free);
                float alpha = 1.f;
                bool rescale = false;
                if (mine0 || mine1) {
                    float m_loc = -INFINITY;
                    if (mine0) m_loc = row_max64(s);
                    if (mine1) m_loc = fmaxf(m_loc, row_max64(s + 64));
                    const float m_cand = m_loc * sl2;
                    const bool need = m_cand > m_ref + kRescaleThreshold;        // true on the first step (m_ref = -inf)
                    rescale = __any_sync(0xffffffffu, need);
                    if (need) {
                        alpha = ex2(m_ref - m_cand);
                        m_ref = m_cand;
                    }
                }
                // probabilities into registers first: the previous step's P V has this long to finish
                float sum0 = 0.f, sum1 = 0.f;
                const float neg_m = -m_ref;
                if (mine0) exp_pack(s, neg_m, sum0, sum1);
                if (mine1) exp_pack(s + 64, neg_m, sum0, sum1);
                // the previous step's P V must be complete before its probabilities are overwritten or O is touched
                if (grp_n > 0) {
                    ok = mbar_wait(&ctl->pv_done, (grp_n - 1) & 1u, ctl, p.status, 32);
                    if (!ok) break;
                    tc_fence_after();
                }
                if (__builtin_expect(pend_out, 0)) write_out();      // warp-uniform: the previous tile's accumulator is complete
                if (__builtin_expect(rescale && o_dirty, 0)) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float o[16];
                        tmem_ld16(lane_addr + kColO + c * 16, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int t = 0; t < 16; t += 2) fmul2(o[t], o[t + 1], alpha);
                        tmem_st16(lane_addr + kColO + c * 16, reinterpret_cast<unsigned*>(o));
                    }
                }
                if (mine0) tmem_st32(lane_addr + kColP, reinterpret_cast<unsigned*>(s));
                else tmem_st32_zero(lane_addr + kColP);
                if (cnt > 1) {
                    if (mine1) tmem_st32(lane_addr + kColP + 32, reinterpret_cast<unsigned*>(s + 64));
                    else tmem_st32_zero(lane_addr + kColP + 32);
                }
                l_sum = l_sum * alpha + (sum0 + sum1);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&ctl->p_full);
                ++grp_n;
                o_dirty = true;
            }
            if (!ok) break;
            if (flags & kSegLast) {
                // -------------------------------------------------------- end of the tile: lse, output pointer
                const int my_q = lower ? slot->qb : slot->qa;
                const unsigned long long qbits = lower ? slot->qbits_b : slot->qbits_a;
                const bool have = live && o_dirty;
                const int part_slot = slot->part_slot;
                if (part_slot >= 0) {
                    // one part of a split tile: (max, sum) now, the accumulator once its last P V is complete
                    float* part = p.partials + (size_t)part_slot * kPartialFloats;
                    part[128 * 64 + row] = have ? m_ref : -INFINITY;
                    part[128 * 64 + 128 + row] = have ? l_sum : 0.f;
                    if (have) {
                        pend_out = true;
                        pend_partial = true;
                        pend_dst = reinterpret_cast<uint4*>(part + row * 64);
                    }
                } else if (my_q >= 0) {                 // warp-uniform
                    const int r64 = row & (kBlock - 1);
                    const bool good = have && ((qbits >> r64) & 1ull) && l_sum > 0.f;
                    const size_t tok = ((size_t)slot->bh * p.nb + my_q) * kBlock + r64;
                    uint4* dst = reinterpret_cast<uint4*>(p.out + tok * kBlock);
                    if (p.lse) p.lse[tok] = good ? (m_ref + __log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
                    if (have) {
                        // the accumulator is read once the tile's last P V is known to be complete
                        pend_out = true;
                        pend_partial = false;
                        pend_inv = good ? __frcp_rn(l_sum) : 0.f;
                        pend_dst = dst;
                    } else {
                        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                        for (int j = 0; j < 8; ++j) dst[j] = z;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&ctl->sched_empty[ss]);
            ++sched_n;
        }
    }

    // ------------------------------------------------------------------------------------------------ teardown
    __syncthreads();
    if (*(volatile int*)&ctl->abort_flag) {
        // a wait expired: give copies and MMAs still in flight time to land before shared and tensor memory go away
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (threadIdx.x == 0) {
        // the last CTA to finish re-arms the work counter for the next launch
        __threadfence();
        const int done = atomicAdd(&p.counter[1], 1);
        if (done == (int)gridDim.x - 1) {
            p.counter[0] = 0;
            p.counter[1] = 0;
            __threadfence();
        }
    }
}

// Combines the parts of the split tiles: one CTA per (batch*head, split tile, group of 16 rows); 16 threads share
// a row, each owning 4 of its 64 output columns.
__global__ void __launch_bounds__(256)
merge_split_tiles_kernel(const float* __restrict__ partials, const int* __restrict__ tile_q, const unsigned long long* __restrict__ kbits,
                         __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int H, int nb, int tiles_per_head, int nparts) {
    const int rgrp = blockIdx.x & 7, tile = (blockIdx.x >> 3) % tiles_per_head, bh = (blockIdx.x >> 3) / tiles_per_head;
    const int row = rgrp * 16 + (threadIdx.x >> 4), c4 = threadIdx.x & 15, r64 = row & (kBlock - 1);
    const int q = tile_q[2 * tile + (row >> 6)];
    if (q < 0) return;
    const unsigned long long qb = kbits ? kbits[(size_t)(bh / H) * nb + q] : ~0ull;
    const float* base = partials + (size_t)(bh * tiles_per_head + tile) * nparts * kPartialFloats;
    float m = -INFINITY;
    for (int pt = 0; pt < nparts; ++pt) m = fmaxf(m, base[(size_t)pt * kPartialFloats + 128 * 64 + row]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    if (m > -INFINITY) {
        for (int pt = 0; pt < nparts; ++pt) {            // fixed order: results do not depend on scheduling
            const float* part = base + (size_t)pt * kPartialFloats;
            const float lp = part[128 * 64 + 128 + row];
            if (!(lp > 0.f)) continue;
            const float wgt = exp2f(part[128 * 64 + row] - m);
            l += wgt * lp;
            const float4 v = reinterpret_cast<const float4*>(part + row * 64)[c4];
            acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
        }
    }
    const bool good = ((qb >> r64) & 1ull) && l > 0.f;
    const float inv = good ? 1.f / l : 0.f;
    const size_t tok = ((size_t)bh * nb + q) * kBlock + r64;
    uint2 v2;
    v2.x = pack_bf16(acc.x * inv, acc.y * inv);
    v2.y = pack_bf16(acc.z * inv, acc.w * inv);
    reinterpret_cast<uint2*>(out + tok * kBlock)[c4] = v2;
    if (lse && c4 == 0) lse[tok] = good ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever arrives on, with the same
// helper and the same limit as the attention kernel; the wait gives up, records BIGBIRD_ETIMEOUT and the kernel
// returns normally.
__global__ void wait_expiry_selftest_kernel(int* status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + kSmemCtl);
    if (threadIdx.x == 0) {
        mbar_init(&ctl->s_full, 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(&ctl->s_full, 0u, ctl, status, 99);
    }
}

// One 64-bit word per (batch, key block): bit t = key_padding_mask[batch, block*64 + t] != 0.
__global__ void pack_mask_kernel(const uint8_t* __restrict__ kpm, unsigned long long* __restrict__ kbits, int n_words) {
    const int word = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (word >= n_words) return;
    const uint8_t* src = kpm + (size_t)word * kBlock;
    const unsigned lo = __ballot_sync(0xffffffffu, src[lane] != 0);
    const unsigned hi = __ballot_sync(0xffffffffu, src[lane + 32] != 0);
    if (lane == 0) kbits[word] = ((unsigned long long)hi << 32) | lo;
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)sym;
    });
    return fn;
}

// [rows, 64] bf16 row-major tensor read in 64 x 64 boxes with the 128-byte swizzle.
bool make_map(CUtensorMap* tm, const void* base, uint64_t rows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kBlock, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)(kBlock * 2)};
    cuuint32_t box[2] = {(cuuint32_t)kBlock, (cuuint32_t)kBlock};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_wait_expiry_selftest(DeviceScratch& sc, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(wait_expiry_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    wait_expiry_selftest_kernel<<<1, 32, kSmemBytes, stream>>>(sc.status);
    return cudaGetLastError();
}

int launch_attn_fwd_sm100(const FwdArgs& a, const bigbird_layout& L, const DeviceLayout& dl, DeviceScratch& sc,
                          int* launches, cudaError_t* cuda_err) {
    *cuda_err = cudaSuccess;
    if (!(a.scale > 0.f) || !(a.scale < INFINITY)) return BIGBIRD_EINVAL;
    const int64_t rows = (int64_t)a.B * a.H * a.N;
    if (rows >= (1ll << 31) || (int64_t)a.B * a.H * L.items_per_head >= (1ll << 31)) return BIGBIRD_EUNSUPPORTED;

    static std::once_flag attr_once;
    static cudaError_t attr_err = cudaSuccess;
    static int sm_count = 0;
    std::call_once(attr_once, [] {
        attr_err = cudaFuncSetAttribute(attn_fwd_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        int dev = 0;
        if (attr_err == cudaSuccess) attr_err = cudaGetDevice(&dev);
        if (attr_err == cudaSuccess) attr_err = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    });
    if (attr_err != cudaSuccess) { *cuda_err = attr_err; return BIGBIRD_ECUDA; }

    CUtensorMap tm_q, tm_k, tm_v;
    if (!make_map(&tm_q, a.q, (uint64_t)rows) || !make_map(&tm_k, a.k, (uint64_t)rows) || !make_map(&tm_v, a.v, (uint64_t)rows)) {
        *cuda_err = cudaErrorInvalidValue;
        return BIGBIRD_ECUDA;
    }

    const unsigned long long* kbits = nullptr;
    if (a.kpm) {
        const size_t words = (size_t)a.B * a.nb;
        if (words > sc.kbits_cap) {                      // grows only when a larger B * N/b shows up
            cudaFree(sc.kbits);
            sc.kbits = nullptr;
            sc.kbits_cap = 0;
            cudaError_t e = cudaMalloc(&sc.kbits, words * sizeof(unsigned long long));
            if (e != cudaSuccess) { *cuda_err = e; return BIGBIRD_ECUDA; }
            sc.kbits_cap = words;
        }
        const int threads = 256, blocks = (int)((words * 32 + threads - 1) / threads);
        pack_mask_kernel<<<blocks, threads, 0, a.stream>>>(a.kpm, sc.kbits, (int)words);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { *cuda_err = e; return BIGBIRD_ECUDA; }
        ++*launches;
        kbits = sc.kbits;
    }

    const bool split = L.split_tiles_per_head > 0 && L.max_parts > 1;
    if (split) {
        const size_t need = (size_t)a.B * a.H * L.split_tiles_per_head * L.max_parts * kPartialFloats;
        if (need > sc.partials_cap) {                    // grows only when a larger problem shows up
            cudaFree(sc.partials);
            sc.partials = nullptr;
            sc.partials_cap = 0;
            cudaError_t e = cudaMalloc(&sc.partials, need * sizeof(float));
            if (e != cudaSuccess) { *cuda_err = e; return BIGBIRD_ECUDA; }
            sc.partials_cap = need;
        }
    }

    KernelParams p{};
    p.out = (__nv_bfloat16*)a.out;
    p.lse = a.lse;
    p.kbits = kbits;
    p.partials = split ? sc.partials : nullptr;
    p.split_tiles_per_head = L.split_tiles_per_head;
    p.max_parts = L.max_parts;
    p.items = dl.items;
    p.steps = dl.steps;
    p.counter = sc.counters + 2 * (sc.next_slot++ % kCounterSlots);
    p.status = sc.status;
    p.items_per_head = L.items_per_head;
    p.heavy_per_head = L.heavy_items_per_head;
    p.BH = a.B * a.H;
    p.H = a.H;
    p.nb = a.nb;
    p.total_work = p.BH * L.items_per_head;
    p.scale_log2 = a.scale * 1.4426950408889634f;

    int grid = 2 * sm_count;
    if (grid > p.total_work) grid = p.total_work;
    if (grid < 1) grid = 1;
    attn_fwd_sm100_kernel<<<grid, kThreads, kSmemBytes, a.stream>>>(tm_q, tm_k, tm_v, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { *cuda_err = e; return BIGBIRD_ECUDA; }
    ++*launches;
    if (split) {
        merge_split_tiles_kernel<<<p.BH * L.split_tiles_per_head * 8, 256, 0, a.stream>>>(sc.partials, dl.split_tile_q, kbits, p.out, p.lse, a.H,
                                                                                     a.nb, L.split_tiles_per_head, L.max_parts);
        e = cudaGetLastError();
        if (e != cudaSuccess) { *cuda_err = e; return BIGBIRD_ECUDA; }
        ++*launches;
    }
    return BIGBIRD_OK;
}

}  // namespace bigbird

// ------------------------------------------------------------------------------------------------ no-allocation entry point
// bigbird_attn_fwd_static: the tensor-core forward for callers that must not allocate device memory (see
// include/bigbird.h).  Everything bigbird_attn_fwd keeps in cudaMalloc'ed library scratch lives here in one
// fixed array that is part of the loaded module: status and work-counter words, the packed key-padding bits,
// and the device copy of the layout's tile schedule, which is re-sent on every call.
namespace bigbird {
namespace {

constexpr size_t kStaticMaskWords = 16384;      // B * N/b
constexpr size_t kStaticItems = 8192;           // H * tiles per head
constexpr size_t kStaticSteps = 131072;         // (key block, halves) entries summed over heads
constexpr size_t kStaticOffMask = 256;          // bytes 0..15: status[2], counter[2]
constexpr size_t kStaticOffItems = kStaticOffMask + kStaticMaskWords * sizeof(unsigned long long);
constexpr size_t kStaticOffSteps = kStaticOffItems + kStaticItems * sizeof(Item);
constexpr size_t kStaticBytes = kStaticOffSteps + kStaticSteps * sizeof(Step);      // about 1.4 MB per GPU

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

struct StaticDevice {
    unsigned char* base = nullptr;              // device address of g_static_scratch on this device
    int sm_count = 0;
};
std::mutex g_static_mu;
StaticDevice g_static_dev[64];

// Once per device, with that device current: the device address of the array (its name is only a host-side
// stand-in in host code) and the kernel's shared-memory attribute.
cudaError_t static_setup(int device, StaticDevice* out) {
    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticDevice& d = g_static_dev[device];
    if (!d.base) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(attn_fwd_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        d.sm_count = sms;
        d.base = (unsigned char*)ptr;
    }
    *out = d;
    return cudaSuccess;
}

}  // namespace
}  // namespace bigbird

extern "C" int bigbird_attn_fwd_static(const void* q, const void* k, const void* v, const bigbird_layout* L,
                                       const uint8_t* key_padding_mask, void* out, float* lse, int B, int H, int64_t N,
                                       int D, int b, float scale, int dtype, void* stream_) {
    using namespace bigbird;
    if (!q || !k || !v || !L || !out) return BIGBIRD_EINVAL;
    if (B < 1 || H < 1 || N < 1 || D < 1 || b < 1) return BIGBIRD_EINVAL;
    if (L->N != N || L->b != b || L->H != H) return BIGBIRD_EINVAL;
    if (dtype != BIGBIRD_BF16 || D != 64 || b != 64) return BIGBIRD_EUNSUPPORTED;
    if ((((uintptr_t)q) | ((uintptr_t)k) | ((uintptr_t)v) | ((uintptr_t)out)) & 15) return BIGBIRD_EINVAL;
    if (!(scale > 0.f) || !(scale < INFINITY)) return BIGBIRD_EINVAL;
    const int64_t rows = (int64_t)B * H * N;
    if (rows >= (1ll << 31) || (int64_t)B * H * L->items_per_head >= (1ll << 31)) return BIGBIRD_EUNSUPPORTED;
    // the fixed scratch bounds the problem
    const size_t words = (size_t)B * L->nb, n_items = L->items.size(), n_steps = L->steps.size();
    if (words > kStaticMaskWords || n_items > kStaticItems || n_steps > kStaticSteps) return BIGBIRD_ELIMIT;
    if (L->max_parts > 1) return BIGBIRD_ELIMIT;    // split global tiles need scratch for their partial results

    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return BIGBIRD_ECUDA;
    if (device < 0 || device >= 64) return BIGBIRD_EUNSUPPORTED;
    StaticDevice sd;
    if (static_setup(device, &sd) != cudaSuccess) return BIGBIRD_ECUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    int* words4 = reinterpret_cast<int*>(sd.base);
    unsigned long long* kbits_dev = reinterpret_cast<unsigned long long*>(sd.base + kStaticOffMask);
    Item* items_dev = reinterpret_cast<Item*>(sd.base + kStaticOffItems);
    Step* steps_dev = reinterpret_cast<Step*>(sd.base + kStaticOffSteps);

    CUtensorMap tm_q, tm_k, tm_v;
    if (!make_map(&tm_q, q, (uint64_t)rows) || !make_map(&tm_k, k, (uint64_t)rows) || !make_map(&tm_v, v, (uint64_t)rows))
        return BIGBIRD_ECUDA;

    // The array keeps what the last call left: status and work counter must start at zero, and the schedule of
    // this call's layout replaces the previous one (step offsets made absolute, as the kernel expects).
    e = cudaMemsetAsync(words4, 0, 16, stream);
    if (e != cudaSuccess) return BIGBIRD_ECUDA;
    static thread_local std::vector<Item> items_abs;            // host memory only
    items_abs = L->items;
    for (int h = 0; h < L->H; ++h)
        for (int i = 0; i < L->items_per_head; ++i) items_abs[(size_t)h * L->items_per_head + i].step_begin += L->step_base[h];
    e = cudaMemcpyAsync(items_dev, items_abs.data(), n_items * sizeof(Item), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && n_steps) e = cudaMemcpyAsync(steps_dev, L->steps.data(), n_steps * sizeof(Step), cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return BIGBIRD_ECUDA;

    const unsigned long long* kbits = nullptr;
    if (key_padding_mask) {
        const int threads = 256, blocks = (int)((words * 32 + threads - 1) / threads);
        pack_mask_kernel<<<blocks, threads, 0, stream>>>(key_padding_mask, kbits_dev, (int)words);
        if (cudaGetLastError() != cudaSuccess) return BIGBIRD_ECUDA;
        kbits = kbits_dev;
    }

    KernelParams p{};
    p.out = (__nv_bfloat16*)out;
    p.lse = lse;
    p.kbits = kbits;
    p.items = items_dev;
    p.steps = steps_dev;
    p.status = words4;
    p.counter = words4 + 2;
    p.items_per_head = L->items_per_head;
    p.heavy_per_head = L->heavy_items_per_head;
    p.BH = B * H;
    p.H = H;
    p.nb = L->nb;
    p.total_work = p.BH * L->items_per_head;
    p.scale_log2 = scale * 1.4426950408889634f;
    int grid = 2 * sd.sm_count;
    if (grid > p.total_work) grid = p.total_work;
    if (grid < 1) grid = 1;
    attn_fwd_sm100_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, p);
    if (cudaGetLastError() != cudaSuccess) return BIGBIRD_ECUDA;
    return BIGBIRD_OK;
}
