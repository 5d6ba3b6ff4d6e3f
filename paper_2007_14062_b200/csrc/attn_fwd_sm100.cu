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
constexpr int kThreads = 192;              // warp 0 producer, warp 1 MMA issuer, warps 2..5 softmax
constexpr int kSoftmaxWarps = 4;
constexpr int kTmemCols = 256;
constexpr int kColS = 0;                   // scores: 2 x 64 fp32 columns
constexpr int kColP = 128;                 // probabilities: 2 x 32 columns of packed bf16 pairs
constexpr int kColO = 192;                 // output accumulator: 64 fp32 columns
constexpr float kRescaleThreshold = 8.0f;  // in log2 units
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct __align__(8) SmemCtl {
    unsigned long long full[kRingSlots];
    unsigned long long empty[kRingSlots];
    unsigned long long q_full, q_empty;
    unsigned long long s_full, s_free, p_full, pv_done;
    unsigned long long sched_full[2], sched_empty[2];
    int work[2];
    unsigned tmem_base;
    int abort_flag;
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
__device__ __noinline__ bool mbar_wait_slow(unsigned long long* bar, unsigned parity, SmemCtl* ctl, int* status, int code) {
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

__device__ __forceinline__ void tmem_ld64(unsigned taddr, float* r) {
    unsigned* u = reinterpret_cast<unsigned*>(r);
#define BB_R(i) "=r"(u[i])
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
        "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
        "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : BB_R(0), BB_R(1), BB_R(2), BB_R(3), BB_R(4), BB_R(5), BB_R(6), BB_R(7), BB_R(8), BB_R(9), BB_R(10), BB_R(11),
          BB_R(12), BB_R(13), BB_R(14), BB_R(15), BB_R(16), BB_R(17), BB_R(18), BB_R(19), BB_R(20), BB_R(21), BB_R(22),
          BB_R(23), BB_R(24), BB_R(25), BB_R(26), BB_R(27), BB_R(28), BB_R(29), BB_R(30), BB_R(31), BB_R(32), BB_R(33),
          BB_R(34), BB_R(35), BB_R(36), BB_R(37), BB_R(38), BB_R(39), BB_R(40), BB_R(41), BB_R(42), BB_R(43), BB_R(44),
          BB_R(45), BB_R(46), BB_R(47), BB_R(48), BB_R(49), BB_R(50), BB_R(51), BB_R(52), BB_R(53), BB_R(54), BB_R(55),
          BB_R(56), BB_R(57), BB_R(58), BB_R(59), BB_R(60), BB_R(61), BB_R(62), BB_R(63)
        : "r"(taddr) : "memory");
#undef BB_R
}
__device__ __forceinline__ void tmem_st32(unsigned taddr, const unsigned* u) {
#define BB_R(i) "r"(u[i])
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::BB_R(0), BB_R(1), BB_R(2), BB_R(3), BB_R(4), BB_R(5), BB_R(6), BB_R(7), BB_R(8), BB_R(9), BB_R(10), BB_R(11),
          BB_R(12), BB_R(13), BB_R(14), BB_R(15), BB_R(16), BB_R(17), BB_R(18), BB_R(19), BB_R(20), BB_R(21), BB_R(22),
          BB_R(23), BB_R(24), BB_R(25), BB_R(26), BB_R(27), BB_R(28), BB_R(29), BB_R(30), BB_R(31), "r"(taddr)
        : "memory");
#undef BB_R
}
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

// ------------------------------------------------------------------------------------------------ schedule helpers
struct Work {
    int bh, h, batch;
    Item item;
};
__device__ __forceinline__ Work decode_work(const KernelParams& p, int w) {
    Work k;
    int it;
    const int heavy_total = p.BH * p.heavy_per_head;
    if (w < heavy_total) {
        k.bh = w / p.heavy_per_head;
        it = w - k.bh * p.heavy_per_head;
    } else {
        const int sparse = p.items_per_head - p.heavy_per_head;
        const int w2 = w - heavy_total;
        k.bh = w2 / sparse;
        it = p.heavy_per_head + (w2 - k.bh * sparse);
    }
    k.h = k.bh % p.H;
    k.batch = k.bh / p.H;
    k.item = p.items[(size_t)k.h * p.items_per_head + it];
    return k;
}
__device__ __forceinline__ unsigned long long key_bits(const KernelParams& p, int batch, int c) {
    if (c < 0) return 0ull;
    return p.kbits ? p.kbits[(size_t)batch * p.nb + c] : ~0ull;
}
// Key blocks of a step that take part: (c0 or -1, c1 or -1); full step: c1 = kStepFull.
struct LiveStep {
    int c0, c1;
    bool full;
    __device__ bool any() const { return c0 >= 0 || c1 >= 0; }
};
__device__ __forceinline__ LiveStep live_step(const KernelParams& p, int batch, Step s, bool has_qb) {
    LiveStep l;
    l.full = s.c1 == kStepFull;
    l.c0 = key_bits(p, batch, s.c0) ? s.c0 : -1;
    l.c1 = (!l.full && has_qb && key_bits(p, batch, s.c1)) ? s.c1 : -1;
    return l;
}
// A tile is skipped when none of its query rows is a real token.
__device__ __forceinline__ bool tile_is_live(const KernelParams& p, const Work& w) {
    if (!p.kbits) return true;
    return (key_bits(p, w.batch, w.item.qa) | key_bits(p, w.batch, w.item.qb)) != 0ull;
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
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->sched_full[i], 1); mbar_init(&ctl->sched_empty[i], 1 + kSoftmaxWarps); }
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

    if (warp == 0) {
        // ===================================================================== producer: scheduler + TMA
        if (lane == 0) {
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
            auto load_step = [&](const CUtensorMap* tm, int bh, const LiveStep& l) -> bool {
                if (l.c0 >= 0 && !load(tm, bh, l.c0)) return false;
                if (l.c1 >= 0 && !load(tm, bh, l.c1)) return false;
                return true;
            };
            while (ok) {
                int w = atomicAdd(&p.counter[0], 1);
                if (w >= p.total_work) w = -1;
                const unsigned ss = sched_n & 1u, sp = (sched_n >> 1) & 1u;
                if (!mbar_wait(&ctl->sched_empty[ss], sp ^ 1u, ctl, p.status, 11)) break;
                ctl->work[ss] = w;
                mbar_arrive(&ctl->sched_full[ss]);      // arrive has release semantics: the store above is visible
                ++sched_n;
                if (w < 0) break;
                const Work wk = decode_work(p, w);
                if (!tile_is_live(p, wk)) continue;
                const bool has_qb = wk.item.qb >= 0;
                // Q tile(s)
                if (!mbar_wait(&ctl->q_empty, (q_n & 1u) ^ 1u, ctl, p.status, 12)) break;
                mbar_expect_tx(&ctl->q_full, has_qb ? 2 * kTileBytes : kTileBytes);
                tma_load_tile(smem + kSmemQ, &tm_q, (wk.bh * p.nb + wk.item.qa) * kBlock, &ctl->q_full);
                if (has_qb) tma_load_tile(smem + kSmemQ + kTileBytes, &tm_q, (wk.bh * p.nb + wk.item.qb) * kBlock, &ctl->q_full);
                ++q_n;
                // K of step i+1 goes ahead of V of step i: the order in which the MMA thread consumes them
                LiveStep prev{-1, -1, false};
                for (int i = 0; i < wk.item.step_count && ok; ++i) {
                    const LiveStep l = live_step(p, wk.batch, p.steps[wk.item.step_begin + i], has_qb);
                    if (!l.any()) continue;
                    ok = load_step(&tm_k, wk.bh, l);
                    if (ok && prev.any()) ok = load_step(&tm_v, wk.bh, prev);
                    prev = l;
                }
                if (ok && prev.any()) ok = load_step(&tm_v, wk.bh, prev);
            }
        }
    } else if (warp == 1) {
        // ===================================================================== MMA issuer
        if (lane == 0) {
            unsigned ring_n = 0, q_n = 0, sched_n = 0, grp_n = 0;     // grp_n: live steps issued so far (QK groups)
            unsigned pv_n = 0;
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
            auto pv_step = [&](const LiveStep& l) -> bool {
                if (!mbar_wait(&ctl->p_full, pv_n & 1u, ctl, p.status, 22)) return false;
                tc_fence_after();
                if (l.c0 >= 0 && !pv(0)) return false;
                if (l.c1 >= 0 && !pv(32)) return false;
                tc_commit(&ctl->pv_done);
                ++pv_n;
                return true;
            };
            while (ok) {
                const unsigned ss = sched_n & 1u, sp = (sched_n >> 1) & 1u;
                if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 23)) break;
                const int w = *(volatile int*)&ctl->work[ss];
                mbar_arrive(&ctl->sched_empty[ss]);
                ++sched_n;
                if (w < 0) break;
                const Work wk = decode_work(p, w);
                if (!tile_is_live(p, wk)) continue;
                const bool has_qb = wk.item.qb >= 0;
                if (!mbar_wait(&ctl->q_full, q_n & 1u, ctl, p.status, 24)) break;
                tc_fence_after();
                LiveStep prev{-1, -1, false};
                for (int i = 0; i < wk.item.step_count && ok; ++i) {
                    const LiveStep l = live_step(p, wk.batch, p.steps[wk.item.step_begin + i], has_qb);
                    if (!l.any()) continue;
                    // the softmax warps must have pulled the previous scores out of tensor memory
                    ok = mbar_wait(&ctl->s_free, (grp_n & 1u) ^ 1u, ctl, p.status, 25);
                    if (!ok) break;
                    tc_fence_after();
                    if (l.c0 >= 0) ok = qk(0);
                    if (ok && l.c1 >= 0) ok = qk(64);
                    if (!ok) break;
                    tc_commit(&ctl->s_full);
                    ++grp_n;
                    if (prev.any()) ok = pv_step(prev);
                    prev = l;
                }
                if (!ok) break;
                tc_commit(&ctl->q_empty);               // every Q K^T of the tile has been issued
                ++q_n;
                if (prev.any()) ok = pv_step(prev);
            }
        }
    } else {
        // ===================================================================== softmax + epilogue (128 threads)
        const int quad = warp & 3;                      // tensor-memory lanes this warp may touch: 32*quad .. +31
        const int row = quad * 32 + lane;               // row of the 128-row tile
        const bool lower = row >= kBlock;
        const unsigned lane_addr = tmem + ((unsigned)(quad * 32) << 16);
        unsigned sched_n = 0, grp_n = 0;
        bool ok = true;
        while (ok) {
            const unsigned ss = sched_n & 1u, sp = (sched_n >> 1) & 1u;
            if (!mbar_wait(&ctl->sched_full[ss], sp, ctl, p.status, 30)) break;
            const int w = *(volatile int*)&ctl->work[ss];
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->sched_empty[ss]);
            ++sched_n;
            if (w < 0) break;
            const Work wk = decode_work(p, w);
            const bool has_qb = wk.item.qb >= 0;
            const int my_q = lower ? wk.item.qb : wk.item.qa;
            const bool live = tile_is_live(p, wk);
            float m_ref = -INFINITY, l_sum = 0.f;
            bool o_dirty = false;                       // has any P V been accumulated for this tile yet
            if (live) {
                // clear the accumulator (the previous tile's epilogue has already read it)
                tmem_st32_zero(lane_addr + kColO);
                tmem_st32_zero(lane_addr + kColO + 32);
                for (int i = 0; i < wk.item.step_count && ok; ++i) {
                    const LiveStep l = live_step(p, wk.batch, p.steps[wk.item.step_begin + i], has_qb);
                    if (!l.any()) continue;
                    const int my_c = l.full ? (my_q >= 0 ? l.c0 : -1) : (lower ? l.c1 : l.c0);   // warp-uniform
                    const int my_half = (l.full || !lower) ? 0 : 1;
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
                        const unsigned long long kb = key_bits(p, wk.batch, my_c);
                        if (kb != ~0ull) {
#pragma unroll
                            for (int j = 0; j < 64; ++j) s[j] = ((kb >> j) & 1ull) ? s[j] : -INFINITY;
                        }
                        float mx = s[0];
#pragma unroll
                        for (int j = 1; j < 64; ++j) mx = fmaxf(mx, s[j]);
                        const float m_cand = mx * p.scale_log2;
                        const bool need = m_cand > m_ref + kRescaleThreshold;    // true on the first step (m_ref = -inf)
                        rescale = __any_sync(0xffffffffu, need);
                        if (need) {
                            alpha = ex2(m_ref - m_cand);
                            m_ref = m_cand;
                        }
                        float sum = 0.f;
#pragma unroll
                        for (int j = 0; j < 64; j += 2) {
                            const float p0 = ex2(fmaf(s[j], p.scale_log2, -m_ref));
                            const float p1 = ex2(fmaf(s[j + 1], p.scale_log2, -m_ref));
                            sum += p0 + p1;
                            pk[j >> 1] = pack_bf16(p0, p1);
                        }
                        l_sum = l_sum * alpha + sum;
                    }
                    // P of the previous step must have been consumed, and O must be at rest, before touching either
                    ok = mbar_wait(&ctl->pv_done, (grp_n & 1u) ^ 1u, ctl, p.status, 32);
                    if (!ok) break;
                    tc_fence_after();
                    if (rescale && o_dirty) {
                        float o[64];
                        tmem_ld64(lane_addr + kColO, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 64; ++j) o[j] *= alpha;
                        tmem_st32(lane_addr + kColO, reinterpret_cast<unsigned*>(o));
                        tmem_st32(lane_addr + kColO + 32, reinterpret_cast<unsigned*>(o) + 32);
                    }
                    if (l.full) {
                        if (my_c >= 0) tmem_st32(lane_addr + kColP, pk);
                        else tmem_st32_zero(lane_addr + kColP);                  // tile without a lower query block
                    } else {
                        // split step: my probabilities go to my half, zeros to the half of the other key block
                        if (my_c >= 0) tmem_st32(lane_addr + kColP + my_half * 32, pk);
                        const int other_c = lower ? l.c0 : l.c1;
                        if (other_c >= 0) tmem_st32_zero(lane_addr + kColP + (1 - (lower ? 1 : 0)) * 32);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->p_full);
                    ++grp_n;
                    o_dirty = true;
                }
                if (!ok) break;
            }
            // ------------------------------------------------------------ epilogue of the tile
            float o[64];
            bool have = false;
            if (live && o_dirty) {
                ok = mbar_wait(&ctl->pv_done, (grp_n & 1u) ^ 1u, ctl, p.status, 33);   // last P V of the tile
                if (!ok) break;
                tc_fence_after();
                tmem_ld64(lane_addr + kColO, o);
                tmem_wait_ld();
                have = true;
            }
            if (my_q >= 0) {
                const int r64 = row & (kBlock - 1);
                const bool q_valid = (key_bits(p, wk.batch, my_q) >> r64) & 1ull;
                const bool good = have && q_valid && l_sum > 0.f;
                const float inv = good ? 1.f / l_sum : 0.f;
                const size_t tok = ((size_t)wk.bh * p.nb + my_q) * kBlock + r64;
                uint4* dst = reinterpret_cast<uint4*>(p.out + tok * kBlock);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint4 v4;
                    v4.x = good ? pack_bf16(o[8 * j + 0] * inv, o[8 * j + 1] * inv) : 0u;
                    v4.y = good ? pack_bf16(o[8 * j + 2] * inv, o[8 * j + 3] * inv) : 0u;
                    v4.z = good ? pack_bf16(o[8 * j + 4] * inv, o[8 * j + 5] * inv) : 0u;
                    v4.w = good ? pack_bf16(o[8 * j + 6] * inv, o[8 * j + 7] * inv) : 0u;
                    dst[j] = v4;
                }
                if (p.lse) p.lse[tok] = good ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
            }
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
