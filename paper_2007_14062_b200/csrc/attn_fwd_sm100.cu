// BigBird block-sparse attention forward on Blackwell tensor cores (sm_100a).
//
// What is computed: Eq. (AT) of arXiv 2007.14062 (softmax attention restricted to the out-neighbours of each
// query) over the block graph of App. D.  How, on B200:
//
//   * Two query blocks are stacked into one 128-row tile so that every tcgen05.mma runs at M = 128.  The
//     tile walks a list of steps prepared on the host: a full step is a key block both halves attend; a split
//     step pairs a key block only the upper half attends with one only the lower half attends.
//   * A producer warp fetches Q once per tile and the K and V blocks of each step with TMA (128-byte swizzle)
//     straight from the [B, H, N, D] tensors into a shared-memory ring: nothing is gathered or packed in HBM.
//   * One thread issues S = Q K^T and O += P V as tcgen05.mma (bf16 operands, fp32 accumulators in tensor
//     memory).  P is handed to the second MMA through tensor memory.
//   * Four softmax warps own one row each per thread: tcgen05.ld of the scores, key-padding mask, running
//     maximum and sum in fp32 (base-2 exponentials), bf16 probabilities written back with tcgen05.st.  The
//     accumulator is rescaled only when the running maximum grows by more than 2^8.
//   * CTAs are persistent and draw work from a global counter: global-row tiles first, then the sparse tiles
//     in (batch, head)-major order.  Two CTAs share an SM so that one's softmax overlaps the other's MMAs.
//
// Every wait on an mbarrier is bounded: on expiry the kernel records BIGBIRD_ETIMEOUT and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "kernels.h"
#include "../../include/bigbird.h"

namespace bigbird {
namespace {

// ------------------------------------------------------------------------------------------------ constants
constexpr int kBlock = 64;                 // tokens per block (b) and head dimension (D)
constexpr int kTileBytes = kBlock * kBlock * 2;      // one 64x64 bf16 tile
constexpr int kRingSlots = 10;
constexpr int kThreads = 256;              // warp 0 TMA, warp 1 MMA issuer, warp 2 scheduler, warp 3 idle, warps 4..7 softmax
constexpr int kSoftmaxWarps = 4;
#ifndef BB_REGS_LIGHT
#define BB_REGS_LIGHT 64
#define BB_REGS_SOFTMAX 192
#endif
constexpr int kRegsLight = BB_REGS_LIGHT;             // registers per thread of warps 0..3 after setmaxnreg
constexpr int kRegsSoftmax = BB_REGS_SOFTMAX;          // registers per thread of warps 4..7 after setmaxnreg
constexpr int kTmemCols = 256;
constexpr int kColS = 0;                   // scores: 2 x 64 fp32 columns
constexpr int kColP = 128;                 // probabilities: 2 x 32 columns of packed bf16 pairs
constexpr int kColO = 192;                 // output accumulator: 64 fp32 columns
constexpr float kRescaleThreshold = 8.0f;  // in log2 units
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr int kSchedSlots = 3;
constexpr int kSegSteps = 64;              // live steps per posted segment of a tile

// A step of a tile after the key-padding mask has been applied: key blocks that are entirely padding are gone.
struct __align__(16) StepEntry {
    int c0, c1;                    // key block of the upper / lower half (or of both when full), -1 = none
    int full;
    int pad_;
    unsigned long long kb0, kb1;   // valid-key bits of c0 / c1
};
enum { kSegFirst = 1, kSegLast = 2, kSegLive = 4 };
struct __align__(16) WorkSlot {
    int w;                         // work index, -1 = no more work
    int bh, batch, qa, qb;
    int n_steps;
    int flags;
    int pad_;
    unsigned long long qbits_a, qbits_b;
    StepEntry steps[kSegSteps];
};

struct __align__(16) SmemCtl {
    unsigned long long full[kRingSlots];
    unsigned long long empty[kRingSlots];
    unsigned long long q_full, q_empty;
    unsigned long long s_full, s_free, p_full, pv_done;
    unsigned long long sched_full[kSchedSlots], sched_empty[kSchedSlots];
    unsigned tmem_base;
    int abort_flag;
    WorkSlot slot[kSchedSlots];
};
constexpr int kSmemQ = 0;
constexpr int kSmemRing = 2 * kTileBytes;
constexpr int kSmemCtl = kSmemRing + kRingSlots * kTileBytes;
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

// Bounded wait.  Returns false if the wait expired or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait_slow(unsigned long long* bar, unsigned parity, SmemCtl* ctl, int* status, int code) {
    const unsigned long long t0 = global_ns();
    for (unsigned it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*(volatile int*)&ctl->abort_flag) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                if (atomicCAS(status, 0, BIGBIRD_ETIMEOUT) == 0) status[1] = code;
                *(volatile int*)&ctl->abort_flag = 1;
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, SmemCtl* ctl, int* status, int code) {
    if (mbar_try(bar, parity)) return true;
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
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 64; B is K-major (K^T) or MN-major (V).
constexpr unsigned kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr unsigned kIdescPV = kIdescQK | (1u << 16);

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

// ------------------------------------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(kThreads, 2)
attn_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const KernelParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + kSmemCtl);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kRingSlots; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], 1); }
        mbar_init(&ctl->q_full, 1);
        mbar_init(&ctl->q_empty, 1);
        mbar_init(&ctl->s_full, 1);
        mbar_init(&ctl->s_free, kSoftmaxWarps);
        mbar_init(&ctl->p_full, kSoftmaxWarps);
        mbar_init(&ctl->pv_done, 1);
        for (int i = 0; i < kSchedSlots; ++i) { mbar_init(&ctl->sched_full[i], 1); mbar_init(&ctl->sched_empty[i], 2 + kSoftmaxWarps); }
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
            // ================================================================= scheduler: fetch work, post live steps
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
                const bool has_qb = item.qb >= 0;
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
                    while (i0 < n_raw && count <= kSegSteps - 32) {
                        const int i = i0 + lane;
                        StepEntry e{-1, -1, 0, 0, 0ull, 0ull};
                        if (i < n_raw) {
                            const Step s = p.steps[item.step_begin + i];
                            e.full = s.c1 == kStepFull;
                            e.kb0 = key_bits(p, batch, s.c0);
                            e.kb1 = (!e.full && has_qb) ? key_bits(p, batch, s.c1) : 0ull;
                            e.c0 = e.kb0 ? s.c0 : -1;
                            e.c1 = e.kb1 ? s.c1 : -1;
                        }
                        const bool alive = e.c0 >= 0 || e.c1 >= 0;
                        const unsigned bal = __ballot_sync(0xffffffffu, alive);
                        if (alive) slot->steps[count + __popc(bal & lt_mask)] = e;
                        count += __popc(bal);
                        i0 += 32;
                    }
                    if (lane == 0) {
                        slot->w = w;
                        slot->bh = bh;
                        slot->batch = batch;
                        slot->qa = item.qa;
                        slot->qb = item.qb;
                        slot->n_steps = count;
                        slot->flags = (first ? kSegFirst : 0) | (i0 >= n_raw ? kSegLast : 0) | (tile_live ? kSegLive : 0);
                        slot->qbits_a = qbits_a;
                        slot->qbits_b = qbits_b;
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
            unsigned ring_n = 0, q_n = 0, sched_n = 0;
            bool ok = true;
            auto load = [&](const CUtensorMap* tm, int bh, int block) -> bool {
                const unsigned slot = ring_n % kRingSlots, ph = (ring_n / kRingSlots) & 1u;
                if (!mbar_wait(&ctl->empty[slot], ph ^ 1u, ctl, p.status, 10)) return false;
                mbar_expect_tx(&ctl->full[slot], kTileBytes);
                tma_load_tile(smem + kSmemRing + slot * kTileBytes, tm, (bh * p.nb + block) * kBlock, &ctl->full[slot]);
                ++ring_n;
                return true;
            };
            auto load_pair = [&](const CUtensorMap* tm, int bh, int c0, int c1) -> bool {
                if (c0 >= 0 && !load(tm, bh, c0)) return false;
                if (c1 >= 0 && !load(tm, bh, c1)) return false;
                return true;
            };
            int prev_c0 = -1, prev_c1 = -1;
            while (ok) {
                const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
                if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 13)) break;
                const WorkSlot* slot = &ctl->slot[ss];
                const int w = slot->w, flags = slot->flags, bh = slot->bh, n = slot->n_steps;
                if (w >= 0 && (flags & kSegLive)) {
                    if (flags & kSegFirst) {
                        const int qa = slot->qa, qb = slot->qb;
                        ok = mbar_wait(&ctl->q_empty, (q_n & 1u) ^ 1u, ctl, p.status, 12);
                        if (!ok) break;
                        mbar_expect_tx(&ctl->q_full, qb >= 0 ? 2 * kTileBytes : kTileBytes);
                        tma_load_tile(smem + kSmemQ, &tm_q, (bh * p.nb + qa) * kBlock, &ctl->q_full);
                        if (qb >= 0) tma_load_tile(smem + kSmemQ + kTileBytes, &tm_q, (bh * p.nb + qb) * kBlock, &ctl->q_full);
                        ++q_n;
                        prev_c0 = prev_c1 = -1;
                    }
                    // K of step i+1 goes ahead of V of step i: the order in which the MMA thread consumes them
                    for (int i = 0; i < n && ok; ++i) {
                        const int c0 = slot->steps[i].c0, c1 = slot->steps[i].c1;
                        ok = load_pair(&tm_k, bh, c0, c1);
                        if (ok) ok = load_pair(&tm_v, bh, prev_c0, prev_c1);
                        prev_c0 = c0;
                        prev_c1 = c1;
                    }
                    if (ok && (flags & kSegLast)) ok = load_pair(&tm_v, bh, prev_c0, prev_c1);
                }
                mbar_arrive(&ctl->sched_empty[ss]);
                ++sched_n;
                if (w < 0) break;
            }
        } else if (warp == 1 && lane == 0) {
            // ================================================================= MMA issuer
            unsigned ring_n = 0, q_n = 0, sched_n = 0, grp_n = 0, pv_n = 0;   // grp_n: live steps whose Q K^T was issued
            bool ok = true;
            const unsigned long long q_desc = smem_desc_sw128(smem_u32(smem + kSmemQ));
            auto qk = [&](int col_off) -> bool {        // S[:, col_off .. col_off+63] = Q K^T with K in the next ring slot
                const unsigned slot = ring_n % kRingSlots, ph = (ring_n / kRingSlots) & 1u;
                if (!mbar_wait(&ctl->full[slot], ph, ctl, p.status, 20)) return false;
                tc_fence_after();
                const unsigned long long k_desc = smem_desc_sw128(smem_u32(smem + kSmemRing + slot * kTileBytes));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)          // 16 head dims (32 bytes inside the swizzled row) per MMA
                    mma_ss(tmem + kColS + col_off, q_desc + (unsigned long long)(kk * 2), k_desc + (unsigned long long)(kk * 2), kIdescQK, kk > 0);
                tc_commit(&ctl->empty[slot]);
                ++ring_n;
                return true;
            };
            auto pv = [&](int p_col_off) -> bool {      // O += P[:, 64 keys] V with V in the next ring slot
                const unsigned slot = ring_n % kRingSlots, ph = (ring_n / kRingSlots) & 1u;
                if (!mbar_wait(&ctl->full[slot], ph, ctl, p.status, 21)) return false;
                tc_fence_after();
                const unsigned long long v_desc = smem_desc_sw128(smem_u32(smem + kSmemRing + slot * kTileBytes));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)          // 16 keys per MMA: 8 packed columns of P, two 8-row groups of V
                    mma_ts(tmem + kColO, tmem + kColP + p_col_off + kk * 8, v_desc + (unsigned long long)(kk * (2048 >> 4)), kIdescPV, 1u);
                tc_commit(&ctl->empty[slot]);
                ++ring_n;
                return true;
            };
            auto pv_step = [&](int c0, int c1) -> bool {
                if (!mbar_wait(&ctl->p_full, pv_n & 1u, ctl, p.status, 22)) return false;
                tc_fence_after();
                if (c0 >= 0 && !pv(0)) return false;
                if (c1 >= 0 && !pv(32)) return false;
                tc_commit(&ctl->pv_done);
                ++pv_n;
                return true;
            };
            int prev_c0 = -1, prev_c1 = -1;
            while (ok) {
                const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
                if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 23)) break;
                const WorkSlot* slot = &ctl->slot[ss];
                const int w = slot->w, flags = slot->flags, n = slot->n_steps;
                if (w >= 0 && (flags & kSegLive)) {
                    if (flags & kSegFirst) {
                        ok = mbar_wait(&ctl->q_full, q_n & 1u, ctl, p.status, 24);
                        if (!ok) break;
                        tc_fence_after();
                        prev_c0 = prev_c1 = -1;
                    }
                    for (int i = 0; i < n && ok; ++i) {
                        const int c0 = slot->steps[i].c0, c1 = slot->steps[i].c1;
                        // the softmax warps must have pulled the previous scores out of tensor memory
                        ok = mbar_wait(&ctl->s_free, (grp_n & 1u) ^ 1u, ctl, p.status, 25);
                        if (!ok) break;
                        tc_fence_after();
                        if (c0 >= 0) ok = qk(0);
                        if (ok && c1 >= 0) ok = qk(64);
                        if (!ok) break;
                        tc_commit(&ctl->s_full);
                        ++grp_n;
                        if (prev_c0 >= 0 || prev_c1 >= 0) ok = pv_step(prev_c0, prev_c1);
                        prev_c0 = c0;
                        prev_c1 = c1;
                    }
                    if (!ok) break;
                    if (flags & kSegLast) {
                        tc_commit(&ctl->q_empty);       // every Q K^T of the tile has been issued
                        ++q_n;
                        if (prev_c0 >= 0 || prev_c1 >= 0) ok = pv_step(prev_c0, prev_c1);
                    }
                }
                mbar_arrive(&ctl->sched_empty[ss]);
                ++sched_n;
                if (w < 0) break;
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        // ===================================================================== softmax + epilogue (128 threads)
        const int quad = warp & 3;                      // tensor-memory lanes this warp may touch: 32*quad .. +31
        const int row = quad * 32 + lane;               // row of the 128-row tile
        const bool lower = row >= kBlock;
        const unsigned lane_addr = tmem + ((unsigned)(quad * 32) << 16);
        const float sl2 = p.scale_log2;
        unsigned sched_n = 0, grp_n = 0;
        bool ok = true;
        float m_ref = -INFINITY, l_sum = 0.f;
        bool o_dirty = false;                           // has any P V been accumulated for this tile yet
        while (ok) {
            const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
            if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 30)) break;
            const WorkSlot* slot = &ctl->slot[ss];
            const int w = slot->w, flags = slot->flags, n = slot->n_steps;
            if (w < 0) break;
            const int my_q = lower ? slot->qb : slot->qa;
            const bool live = flags & kSegLive;
            if (flags & kSegFirst) {
                m_ref = -INFINITY;
                l_sum = 0.f;
                o_dirty = false;
                if (live) {
                    // clear the accumulator (the previous tile's epilogue has already read it)
                    tmem_st32_zero(lane_addr + kColO);
                    tmem_st32_zero(lane_addr + kColO + 32);
                }
            }
            for (int i = 0; i < n && ok; ++i) {
                const StepEntry* e = &slot->steps[i];
                const int full = e->full;
                const int c0 = e->c0, c1 = e->c1;
                const int my_c = full ? (my_q >= 0 ? c0 : -1) : (lower ? c1 : c0);          // warp-uniform
                const int my_half = (full || !lower) ? 0 : 1;
                ok = mbar_wait(&ctl->s_full, grp_n & 1u, ctl, p.status, 31);
                if (!ok) break;
                tc_fence_after();
                float s[64];
                if (my_c >= 0) {
                    tmem_ld64(lane_addr + kColS + my_half * 64, s);
                    tmem_wait_ld();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->s_free);
                unsigned pk[32];
                float alpha = 1.f;
                bool rescale = false;
                if (my_c >= 0) {
                    const unsigned long long kb = my_half ? e->kb1 : e->kb0;
                    if (kb != ~0ull) {
#pragma unroll
                        for (int j = 0; j < 64; ++j) s[j] = ((kb >> j) & 1ull) ? s[j] : -INFINITY;
                    }
                    float mx0 = max3(s[0], s[1], s[2]), mx1 = max3(s[3], s[4], s[5]);
#pragma unroll
                    for (int j = 6; j < 62; j += 4) {
                        mx0 = max3(mx0, s[j], s[j + 1]);
                        mx1 = max3(mx1, s[j + 2], s[j + 3]);
                    }
                    const float m_cand = max3(mx0, mx1, fmaxf(s[62], s[63])) * sl2;
                    const bool need = m_cand > m_ref + kRescaleThreshold;        // true on the first step (m_ref = -inf)
                    rescale = __any_sync(0xffffffffu, need);
                    if (need) {
                        alpha = ex2(m_ref - m_cand);
                        m_ref = m_cand;
                    }
                    float sum0 = 0.f, sum1 = 0.f;
                    const float neg_m = -m_ref;
#pragma unroll
                    for (int j = 0; j < 64; j += 2) {
                        float t0, t1;
                        ffma2(t0, t1, s[j], s[j + 1], sl2, neg_m);
                        const float p0 = ex2(t0), p1 = ex2(t1);
                        fadd2(sum0, sum1, p0, p1);
                        pk[j >> 1] = pack_bf16(p0, p1);
                    }
                    l_sum = l_sum * alpha + (sum0 + sum1);
                }
                // P of the previous step must have been consumed, and O must be at rest, before touching either
                ok = mbar_wait(&ctl->pv_done, (grp_n & 1u) ^ 1u, ctl, p.status, 32);
                if (!ok) break;
                tc_fence_after();
                if (rescale && o_dirty) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        float o[32];
                        tmem_ld32(lane_addr + kColO + half * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; j += 2) fmul2(o[j], o[j + 1], alpha);
                        tmem_st32(lane_addr + kColO + half * 32, reinterpret_cast<unsigned*>(o));
                    }
                }
                if (full) {
                    if (my_c >= 0) tmem_st32(lane_addr + kColP, pk);
                    else tmem_st32_zero(lane_addr + kColP);                      // tile without a lower query block
                } else {
                    // split step: my probabilities go to my half, zeros to the half of the other key block
                    if (my_c >= 0) tmem_st32(lane_addr + kColP + my_half * 32, pk);
                    const int other_c = lower ? c0 : c1;
                    if (other_c >= 0) tmem_st32_zero(lane_addr + kColP + (lower ? 0 : 32));
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->p_full);
                ++grp_n;
                o_dirty = true;
            }
            if (!ok) break;
            if (flags & kSegLast) {
                // -------------------------------------------------------- epilogue of the tile
                const int bh = slot->bh;
                const unsigned long long qbits = lower ? slot->qbits_b : slot->qbits_a;
                const bool have = live && o_dirty;
                if (have) {
                    ok = mbar_wait(&ctl->pv_done, (grp_n & 1u) ^ 1u, ctl, p.status, 33);   // last P V of the tile
                    if (!ok) break;
                    tc_fence_after();
                }
                if (my_q >= 0) {
                    const int r64 = row & (kBlock - 1);
                    const bool good = have && ((qbits >> r64) & 1ull) && l_sum > 0.f;
                    const float inv = good ? 1.f / l_sum : 0.f;
                    const size_t tok = ((size_t)bh * p.nb + my_q) * kBlock + r64;
                    uint4* dst = reinterpret_cast<uint4*>(p.out + tok * kBlock);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        float o[32];
                        if (have) {                     // warp-uniform
                            tmem_ld32(lane_addr + kColO + half * 32, o);
                            tmem_wait_ld();
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 v4;
                            v4.x = good ? pack_bf16(o[8 * j + 0] * inv, o[8 * j + 1] * inv) : 0u;
                            v4.y = good ? pack_bf16(o[8 * j + 2] * inv, o[8 * j + 3] * inv) : 0u;
                            v4.z = good ? pack_bf16(o[8 * j + 4] * inv, o[8 * j + 5] * inv) : 0u;
                            v4.w = good ? pack_bf16(o[8 * j + 6] * inv, o[8 * j + 7] * inv) : 0u;
                            dst[half * 4 + j] = v4;
                        }
                    }
                    if (p.lse) p.lse[tok] = good ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->sched_empty[ss]);
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

    KernelParams p{};
    p.out = (__nv_bfloat16*)a.out;
    p.lse = a.lse;
    p.kbits = kbits;
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
    return BIGBIRD_OK;
}

}  // namespace bigbird
