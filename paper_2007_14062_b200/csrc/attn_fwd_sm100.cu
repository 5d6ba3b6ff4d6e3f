// BigBird block-sparse attention forward on Blackwell tensor cores (sm_100a).
//
// What is computed: Eq. (AT) of arXiv 2007.14062 (softmax attention restricted to the out-neighbours of each
// query) over the block graph of App. D.  How, on B200:
//
//   * Two query blocks are stacked into one 128-row tile so that every tcgen05.mma runs at M = 128.  The tile
//     walks a list of key blocks prepared on the host; each is attended by both halves of the tile or by one.
//     The MMAs always cover all 128 rows; rows that do not attend a key block get probability zero for it.
//   * One CTA per SM runs two independent tile streams side by side.  Each stream owns half of tensor memory
//     (scores 128 | probabilities 64 | output accumulator 64 columns), a Q double buffer and a ring of K / V
//     tiles in shared memory, an MMA-issuing thread and a softmax warpgroup.  Two issuing threads keep the
//     tensor pipe full where one thread's issue rate would not (a 64-wide P V instruction takes the pipe less
//     time than one thread needs to issue the next), and the two softmax warpgroups fill each other's gaps on
//     the special-function unit.
//   * Four lanes of a producer warp (per stream one for Q and K, one for V) fetch Q once per tile and the K and V
//     blocks with TMA (128-byte swizzle) straight from the [B, H, N, D] tensors into the stream's ring: nothing is
//     gathered or packed in HBM.
//   * Key blocks are processed two at a time (one "step").  Their K tiles land in adjacent ring slots, so that
//     S = Q K^T of a step is one N = 128 tcgen05.mma per 16 head dimensions.  O += P V follows with P read
//     from tensor memory.
//   * Softmax warpgroup, one thread per row of the tile: the thread pulls its (up to) 128 scores into registers
//     with tcgen05.ld and hands the score columns back at once, so that the next step's Q K^T runs under this
//     step's exponentials; it applies the key-padding mask, takes the row maximum, exponentiates (base 2, fp32),
//     sums, and writes bf16 probabilities with tcgen05.st (zeros for key blocks its half of the tile does not
//     attend).  The accumulator is rescaled only when the running maximum grows by more than 2^8.
//   * An epilogue warpgroup shared by the two streams takes a finished tile's accumulator out of tensor memory,
//     scales it by 1/l and writes the output rows, while the stream's softmax threads are already on the next tile.
//   * A global-row tile of a long sequence is cut along the keys into parts that are separate work items; each
//     writes its unnormalised accumulator and (max, sum) per row to scratch, and a small merge kernel combines
//     the parts in a fixed order.
//   * CTAs are persistent; a scheduler warp draws work for both streams from a global counter: global-row tiles
//     first, then the sparse tiles in (batch, head)-major order.
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
constexpr int kStreams = 2;                // tile streams per CTA
// warps 0..3 / 4..7: softmax of stream 0 / 1; warps 8..11: epilogue; warp 12: TMA producer; warps 13, 14: MMA issuers
// of stream 0 / 1; warp 15: scheduler
constexpr int kThreads = 512;
constexpr int kWarpEpilogue = 8, kWarpProducer = 12, kWarpMma = 13, kWarpScheduler = 15;
constexpr int kSoftmaxThreads = 128;
// 512 threads start with 128 registers each; the roles then trade.  A sub-partition's registers are shared out
// among its own four warps only (setmaxnreg can hand out no more than those warps gave back): two softmax warps x 200
// (a step's 128 scores plus the loop's temporaries) + an epilogue warp x 56 + a light warp x 56 = 4 x 128 exactly.
// Nothing may spill: a spill here costs a trip to L2, since nearly all of the SM's L1 is configured as shared memory.
#ifndef BB_REGS_SOFTMAX
#define BB_REGS_SOFTMAX 200
#define BB_REGS_EPILOGUE 56
#define BB_REGS_LIGHT 56
#endif
constexpr int kRegsSoftmax = BB_REGS_SOFTMAX, kRegsEpilogue = BB_REGS_EPILOGUE, kRegsLight = BB_REGS_LIGHT;
static_assert(2 * kRegsSoftmax + kRegsEpilogue + kRegsLight <= 4 * 128 && kThreads == 512, "register trade between the four warps of a sub-partition");
constexpr int kTmemCols = 512;
constexpr int kStreamCols = kTmemCols / kStreams;
constexpr int kColS = 0;                   // scores: kStepChunks x 64 fp32 columns
constexpr int kColP = kStepChunks * 64;    // probabilities: kStepChunks x 32 columns of packed bf16 pairs
constexpr int kColO = kColP + kStepChunks * 32;   // output accumulator: 64 fp32 columns
constexpr float kRescaleThreshold = 8.0f;  // in log2 units
constexpr long long kWaitLimitCycles = 4000000000ll;   // about two seconds
constexpr int kSchedSlots = 3;
constexpr int kPartialFloats = 128 * 64 + 2 * 128;   // one part of a split tile: O[128][64], max[128], sum[128]
constexpr int kSegChunks = 96;             // live key blocks per posted segment of a tile (a multiple of kStepChunks)
static_assert(kColO + 64 <= kStreamCols && kSegChunks % kStepChunks == 0, "tensor-memory and segment layout");

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
// What the softmax threads of a stream hand to the epilogue warpgroup at the end of a tile.
enum { kEpiTile = 0, kEpiDone = 1 };
struct __align__(16) EpiMsg {
    int kind;                      // kEpiTile, or kEpiDone: the stream has no more tiles
    int bh, qa, qb;
    int part_slot;
    int pad_[3];
    float inv[kSoftmaxThreads];    // per row: 1 / l, or 0 for a row that must come out as zeros
};

struct __align__(16) StreamCtl {
    unsigned long long full[kRingGroups];
    unsigned long long empty[kRingGroups];
    unsigned long long q_full[2], q_empty[2];
    unsigned long long s_full, s_free, p_full, pv_done;
    unsigned long long o_done, o_free;     // a tile's last P V has completed / the epilogue has taken the accumulator
    unsigned long long epi_full[2];
    unsigned long long sched_full[kSchedSlots], sched_empty[kSchedSlots];
    WorkSlot slot[kSchedSlots];
    EpiMsg epi[2];
};
struct __align__(16) SmemCtl {
    StreamCtl st[kStreams];
    unsigned tmem_base;
    int abort_flag;
};
// per stream: two Q buffers of two tiles each, then the ring
constexpr int kStreamSmemQ = 0;
constexpr int kStreamSmemRing = 4 * kTileBytes;
constexpr int kStreamSmemBytes = kStreamSmemRing + kRingGroups * kGroupBytes;
constexpr int kSmemCtl = kStreams * kStreamSmemBytes;
constexpr int kSmemBytes = kSmemCtl + (int)sizeof(SmemCtl) + 1024;   // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");

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

// Non-blocking test of a phase (for the roles that poll several barriers).
__device__ __forceinline__ bool mbar_test(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait, small enough to sit inline at every site (the kernel's hot code has to fit the SM's instruction
// cache, measured at between 32 and 48 KB: a loop with a clock read and its own give-up code per site did not).  A
// failing try keeps the thread suspended for about 1.4 us on this part (measured); after kWaitTries of them, about
// two seconds, the wait is abandoned.  Returns false then, or as soon as another
// thread of the CTA has given up; the caller leaves its loop and calls give_up with the code of the wait.
constexpr unsigned kWaitTries = 1500000;
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, int* abort_flag) {
    // a phase that is already complete is seen by the plain test in a dozen cycles; try_wait, which may put the
    // thread to sleep, takes a few hundred even then (measured on the MMA thread's time line)
    if (mbar_test(bar, parity)) return true;
#pragma unroll 1
    for (unsigned it = 0; it < kWaitTries; ++it) {
        if (mbar_try(bar, parity)) return true;
        if (*(volatile int*)abort_flag) break;
    }
    return false;
}
// Records BIGBIRD_ETIMEOUT and the code of the abandoned wait (the first one wins) and tells the rest of the CTA.
__device__ __forceinline__ void give_up(int* abort_flag, int* status, int code) {
    if (*(volatile int*)abort_flag == 0) {
        if (atomicCAS(status, 0, BIGBIRD_ETIMEOUT) == 0) status[1] = code;
        *(volatile int*)abort_flag = 1;
    }
}
// Checked build (-DBB_DEBUG): indices that come out of the schedule are tested against their ranges before they are
// used as addresses; a failing check records BIGBIRD_EINTERNAL with its code, tells the CTA to stop, and the access
// is skipped.  Nothing traps.  (The memory checker is not available where this library is developed; small cases
// against the oracle and this build stand in for it.)
#ifdef BB_DEBUG
__device__ __forceinline__ bool debug_check(bool good, int* abort_flag, int* status, int code) {
    if (!good && *(volatile int*)abort_flag == 0) {
        if (atomicCAS(status, 0, BIGBIRD_EINTERNAL) == 0) status[1] = code;
        *(volatile int*)abort_flag = 1;
    }
    return good;
}
#define BB_CHECK(cond, code) debug_check((cond), &ctl->abort_flag, p.status, (code))
#else
#define BB_CHECK(cond, code) true
#endif

// The same bound for a role that polls: tick() is called whenever a round over the role's barriers found nothing
// to do; it backs off (a polling warp that spins takes issue slots from the softmax warps of its sub-partition)
// and returns false once the CTA has given up or the idle time exceeds the limit.
struct IdleClock {
    unsigned n = 0;
    long long t0 = 0;
    __device__ __forceinline__ void reset() { n = 0; }
    __device__ __forceinline__ bool tick(int* abort_flag, int* status, int code, unsigned sleep_ns) {
        ++n;
        if ((n & 15u) == 0u) {
            if (*(volatile int*)abort_flag) return false;
            const long long now = clock64();
            if (n == 16u) t0 = now;
            else if (now - t0 > kWaitLimitCycles) {
                give_up(abort_flag, status, code);
                return false;
            }
        }
        if (sleep_ns) __nanosleep(sleep_ns);
        return true;
    }
};

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

// The same, issued only if enable != 0 (a predicated instruction instead of a branch around it: a lone thread pays
// for every branch it executes with a stall until the target is known).
__device__ __forceinline__ void mma_ts_if(unsigned d_tmem, unsigned a_tmem, unsigned long long b_desc, unsigned idesc, unsigned accumulate, unsigned enable) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(enable) : "memory");
}
__device__ __forceinline__ void tc_commit_if(unsigned long long* bar, unsigned enable) {
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar)), "r"(enable) : "memory");
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

// ------------------------------------------------------------------------------------------------ helpers
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

// Rare paths of the softmax threads.
// -inf over the scores of the padded keys of one key block, in tensor memory.
__device__ __forceinline__ void mask_scores(unsigned taddr, unsigned long long kb) {
#pragma unroll 1
    for (int h = 0; h < 2; ++h) {                   // 32 keys at a time (rolled: a rare path should not take up code space)
        float s[32];
        const unsigned bits = (unsigned)(kb >> (32 * h));
        tmem_ld32(taddr + 32 * h, s);
        tmem_wait_ld();
#pragma unroll
        for (int t = 0; t < 32; ++t) s[t] = ((bits >> t) & 1u) ? s[t] : -INFINITY;
        tmem_st32(taddr + 32 * h, reinterpret_cast<unsigned*>(s));
    }
    tmem_wait_st();
}
// This thread's row of the output accumulator times alpha (the running maximum moved by more than the threshold).
__device__ __forceinline__ void rescale_accumulator(unsigned taddr, float alpha) {
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        float o[16];
        tmem_ld16(taddr + c * 16, o);
        tmem_wait_ld();
#pragma unroll
        for (int t = 0; t < 16; t += 2) fmul2(o[t], o[t + 1], alpha);
        tmem_st16(taddr + c * 16, reinterpret_cast<unsigned*>(o));
    }
}

// What every role needs to know about its stream.
struct StreamRef {
    StreamCtl* sc;
    unsigned char* smem;           // the stream's Q buffers and ring
    unsigned tmem;                 // tensor-memory address of the stream's first column (lane 0)
};

// ------------------------------------------------------------------------------------------------ scheduler (one warp, both streams)
// Fetches the next work item for a stream, drops the key blocks that are entirely padding and posts the live
// list.  Returns the work index (-1: the stream has been told that there is no more work), or -2 after an
// expired wait.
__device__ __forceinline__ int schedule_one(const KernelParams& p, SmemCtl* ctl, StreamCtl* sc, unsigned& sched_n, int lane) {
    const unsigned lt_mask = (1u << lane) - 1u;
    int w = 0;
    if (lane == 0) w = atomicAdd(&p.counter[0], 1);
    w = __shfl_sync(0xffffffffu, w, 0);
    if (w >= p.total_work) w = -1;
    // decode the work index: global-row tiles of every (batch, head) first, then the sparse tiles
    int bh = 0, it = 0, batch = 0;
    Item item{};
    if (w >= 0) {
        const int heavy_total = p.BH * p.heavy_per_head;
        const bool heavy = w < heavy_total;
        const unsigned per_head = heavy ? p.heavy_per_head : p.items_per_head - p.heavy_per_head;
        const unsigned x = heavy ? w : w - heavy_total;
        bh = (int)(x / per_head);                   // (one division for either kind of item: this code is kept small)
        it = (int)(x - bh * per_head) + (heavy ? 0 : p.heavy_per_head);
        batch = (int)((unsigned)bh / (unsigned)p.H);
        if (BB_CHECK(bh >= 0 && bh < p.BH && it >= 0 && it < p.items_per_head, 71)) item = p.items[(size_t)(bh - batch * p.H) * p.items_per_head + it];
        else w = -1;
        if (!BB_CHECK(item.step_count >= 0 && item.step_begin >= 0 && item.qa >= 0 && item.qa < p.nb && item.qb < p.nb, 72)) w = -1;
    }
    const unsigned long long qbits_a = w >= 0 ? key_bits(p, batch, item.qa) : 0ull;
    const unsigned long long qbits_b = w >= 0 ? key_bits(p, batch, item.qb) : 0ull;
    const bool tile_live = (qbits_a | qbits_b) != 0ull;      // a tile whose query rows are all padding is skipped
    const int n_raw = (w >= 0 && tile_live) ? item.step_count : 0;
    int i0 = 0;
    bool first = true;
    do {
        const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
        // the first slot of an item is known to be free (the caller tested it); later segments of a long tile wait here
        if (!mbar_wait(&sc->sched_empty[ss], sp ^ 1u, &ctl->abort_flag)) { give_up(&ctl->abort_flag, p.status, 11); return -2; }
        WorkSlot* slot = &sc->slot[ss];
        int count = 0;
#pragma unroll 1
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
                if (!BB_CHECK(s.c >= 0 && s.c < p.nb && (unsigned)s.who <= (unsigned)kLowerHalf, 70)) alive = false;
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
        if (lane == 0) mbar_arrive(&sc->sched_full[ss]);
        ++sched_n;
        first = false;
    } while (i0 < n_raw);
    return w;
}

__device__ __forceinline__ void scheduler_role(const KernelParams& p, SmemCtl* ctl, int lane) {
    unsigned sched_n0 = 0, sched_n1 = 0;            // slots posted per stream (scalars: an indexed array would live in local memory)
    unsigned done = 0;                              // bit s: stream s has been told that there is no more work
    IdleClock idle;
    while (done != (1u << kStreams) - 1u) {
        bool progress = false;
#pragma unroll 1
        for (int s = 0; s < kStreams; ++s) {        // (not unrolled: one copy of the code)
            if ((done >> s) & 1u) continue;
            StreamCtl* sc = &ctl->st[s];
            unsigned n = s == 0 ? sched_n0 : sched_n1;
            const unsigned ss = n % kSchedSlots, sp = (n / kSchedSlots) & 1u;
            if (!__all_sync(0xffffffffu, mbar_test(&sc->sched_empty[ss], sp ^ 1u))) continue;
            const int w = schedule_one(p, ctl, sc, n, lane);
            if (s == 0) sched_n0 = n; else sched_n1 = n;
            if (w == -2) return;
            if (w < 0) done |= 1u << s;
            progress = true;
        }
        if (progress) idle.reset();
        else if (!__all_sync(0xffffffffu, idle.tick(&ctl->abort_flag, p.status, 12, 400))) return;
    }
}

// ------------------------------------------------------------------------------------------------ TMA producer (two lanes per stream)
// Four lanes of the producer warp: per stream one fetches Q and the K blocks, the other the V blocks.  The ring
// order of a stream is the order in which its MMA thread consumes groups, K0 K1 V0 K2 V1 K3 ...: the K blocks of
// step t go to ring entry 2t - 1 (0 for t = 0), its V blocks to entry 2t + 2, so the two lanes never need to talk.
// A lane cannot block (it shares its warp with the others): it polls, backing off briefly between rounds.
__device__ __forceinline__ bool poll_wait(unsigned long long* bar, unsigned parity, IdleClock& idle, int* abort_flag, int* status, int code) {
    while (!mbar_test(bar, parity))
        if (!idle.tick(abort_flag, status, code, 20)) return false;
    idle.reset();
    return true;
}

__device__ __forceinline__ void producer_role(const KernelParams& p, SmemCtl* ctl, const StreamRef& sr, bool v_lane,
                                              const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_v) {
    StreamCtl* sc = sr.sc;
    int* abort_flag = &ctl->abort_flag;
    const CUtensorMap* tm = v_lane ? tm_v : tm_k;
    unsigned sched_n = 0, q_n = 0, step_n = 0;      // step_n: steps of this stream seen so far
    IdleClock idle;
    for (;;) {
        const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
        if (!poll_wait(&sc->sched_full[ss], sp, idle, abort_flag, p.status, 13)) return;
        const WorkSlot* slot = &sc->slot[ss];
        const int w = slot->w, flags = slot->flags, bh = slot->bh, n = slot->n_chunks;
        if (w >= 0 && (flags & kSegLive)) {
            if (!v_lane && (flags & kSegFirst)) {
                const int qa = slot->qa, qb = slot->qb;
                const unsigned qs = q_n & 1u;
                if (!poll_wait(&sc->q_empty[qs], ((q_n >> 1) & 1u) ^ 1u, idle, abort_flag, p.status, 12)) return;
                mbar_expect_tx(&sc->q_full[qs], qb >= 0 ? 2 * kTileBytes : kTileBytes);
                tma_load_tile(sr.smem + kStreamSmemQ + qs * 2 * kTileBytes, tm_q, (bh * p.nb + qa) * kBlock, &sc->q_full[qs]);
                if (qb >= 0) tma_load_tile(sr.smem + kStreamSmemQ + qs * 2 * kTileBytes + kTileBytes, tm_q, (bh * p.nb + qb) * kBlock, &sc->q_full[qs]);
                ++q_n;
            }
            for (int i = 0; i < n; i += kStepChunks) {
                const int cnt = min(kStepChunks, n - i);
                const unsigned ring_i = v_lane ? 2u * step_n + 2u : (step_n == 0u ? 0u : 2u * step_n - 1u);
                const unsigned g = ring_i % kRingGroups, ph = (ring_i / kRingGroups) & 1u;
                const int c0 = slot->chunks[i].c, c1 = cnt > 1 ? slot->chunks[i + 1].c : 0;
                if (!BB_CHECK(bh >= 0 && bh < p.BH && c0 >= 0 && c0 < p.nb && c1 >= 0 && c1 < p.nb && n <= kSegChunks, 73)) return;
                if (!poll_wait(&sc->empty[g], ph ^ 1u, idle, abort_flag, p.status, 10)) return;
                mbar_expect_tx(&sc->full[g], cnt * kTileBytes);
                tma_load_tile(sr.smem + kStreamSmemRing + g * kGroupBytes, tm, (bh * p.nb + c0) * kBlock, &sc->full[g]);
                if (cnt > 1) tma_load_tile(sr.smem + kStreamSmemRing + g * kGroupBytes + kTileBytes, tm, (bh * p.nb + c1) * kBlock, &sc->full[g]);
                ++step_n;
            }
        }
        mbar_arrive(&sc->sched_empty[ss]);
        ++sched_n;
        if (w < 0) return;
    }
}

// ------------------------------------------------------------------------------------------------ MMA issuer (one thread per stream)
// One thread per stream walks the posted slots; a round issues S = Q K^T of a step and, behind it, O += P V of the
// step before (whose probabilities the softmax threads were writing meanwhile).  The thread is alone in its warp, so
// nothing hides its latencies: every branch stalls it until the target is known and every barrier test is a round
// trip to shared memory.  Hence the shape of the loop: the two barriers a product needs are tested back to back and
// one branch takes the combined result; a second key block and the end of a tile are predicated instructions.
// Ring entries (see the producer): the K blocks of step t sit in entry 2t - 1 (0 for t = 0), its V blocks in 2t + 2.
__device__ __forceinline__ void mma_role(const KernelParams& p, SmemCtl* ctl, const StreamRef& sr) {
    StreamCtl* sc = sr.sc;
    int* abort_flag = &ctl->abort_flag;
    unsigned q_n = 0, sched_n = 0, grp_n = 0, pv_n = 0, tile_n = 0;   // grp_n: steps whose Q K^T was issued; tile_n: tiles handed to the epilogue
    int fail = 0;                               // code of the wait that was abandoned, if any
    unsigned pend_cnt = 0;                      // key blocks of the step whose P V is still to be issued (0: none)
    bool pend_fresh = false;                    // ... it is the first of its tile: it overwrites O
    bool pend_last = false;                     // ... the last of its tile: the accumulator is complete after it
    bool tile_steps = false;                    // the current tile has had a step
    const unsigned q_base = smem_u32(sr.smem + kStreamSmemQ), ring_base = smem_u32(sr.smem + kStreamSmemRing);
    // both barriers at once; the blocking waits only if one of them is not there yet
    auto wait2 = [&](unsigned long long* b1, unsigned par1, bool need1, int code1, unsigned long long* b2, unsigned par2, int code2) -> bool {
        const bool t1 = mbar_test(b1, par1), t2 = mbar_test(b2, par2);
        if (__builtin_expect((t1 || !need1) && t2, 1)) return true;
        if (need1 && !mbar_wait(b1, par1, abort_flag)) { fail = code1; return false; }
        if (!mbar_wait(b2, par2, abort_flag)) { fail = code2; return false; }
        return true;
    };
    for (;;) {
        const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
        if (!mbar_wait(&sc->sched_full[ss], sp, abort_flag)) { fail = 23; break; }
        const WorkSlot* slot = &sc->slot[ss];
        const int w = slot->w, flags = slot->flags, n = slot->n_chunks;
        const bool work = w >= 0 && (flags & kSegLive);
        const bool first = work && (flags & kSegFirst), last = work && (flags & kSegLast);
        if (first) {
            tile_steps = false;
            ++q_n;                              // this tile's Q sits in buffer (q_n - 1) & 1
            if (!mbar_wait(&sc->q_full[(q_n - 1) & 1u], ((q_n - 1) >> 1) & 1u, abort_flag)) { fail = 24; break; }
        }
        const unsigned qs = (q_n - 1) & 1u;
        const unsigned long long q_desc = smem_desc_sw128(q_base + qs * 2 * kTileBytes);
        // one round per step of the slot; the slot that says "no more work" gets one round without a Q K^T, which
        // issues the very last P V
        const int n_rounds = work ? (n + kStepChunks - 1) / kStepChunks : (w < 0 ? 1 : 0);
        bool tile_fresh = first;
#pragma unroll 1
        for (int r = 0; r < n_rounds; ++r) {
            const unsigned cnt = work ? (unsigned)min(kStepChunks, n - r * kStepChunks) : 0u;
            if (cnt) {
                // S[:, 0 .. 64 cnt) = Q K^T: the softmax threads must have pulled the previous scores out of tensor
                // memory, and the K blocks must have landed
                const unsigned ring_i = grp_n == 0u ? 0u : 2u * grp_n - 1u;
                const unsigned g = ring_i % kRingGroups, ph = (ring_i / kRingGroups) & 1u;
                // the blocks of a group are adjacent: their 64 cnt rows form one K-major operand
                const unsigned long long k_desc = smem_desc_sw128(ring_base + g * kGroupBytes);
                const unsigned idesc = kIdescQK64 + ((cnt - 1u) << 20);                    // N = 64 cnt
                if (!wait2(&sc->s_free, (grp_n - 1u) & 1u, grp_n > 0u, 25, &sc->full[g], ph, 20)) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)  // 16 head dims (32 bytes inside the swizzled row) per MMA
                    mma_ss(sr.tmem + kColS, q_desc + (unsigned long long)(kk * 2), k_desc + (unsigned long long)(kk * 2), idesc, kk > 0);
                tc_commit(&sc->s_full);
                tc_commit(&sc->empty[g]);
                ++grp_n;
            }
            if (pend_cnt) {
                // O (+)= sum_j P_j V_j with the V blocks of the pending step
                const unsigned ring_i = 2u * pv_n + 2u;
                const unsigned g = ring_i % kRingGroups, ph = (ring_i / kRingGroups) & 1u;
                const unsigned long long v_desc = smem_desc_sw128(ring_base + g * kGroupBytes);
                const unsigned acc0 = pend_fresh ? 0u : 1u, two = pend_cnt > 1u ? 1u : 0u;
                // the epilogue must have taken the previous tile's accumulator before this tile's first P V overwrites it
                if (pend_fresh && tile_n > 0 && !mbar_wait(&sc->o_free, (tile_n - 1) & 1u, abort_flag)) { fail = 27; break; }
                if (!wait2(&sc->p_full, pv_n & 1u, true, 22, &sc->full[g], ph, 21)) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)  // 16 keys per MMA: 8 packed columns of P_j, two 8-row groups of V_j
                    mma_ts(sr.tmem + kColO, sr.tmem + kColP + kk * 8, v_desc + (unsigned long long)((kk * 2048) >> 4), kIdescPV, kk > 0 ? 1u : acc0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts_if(sr.tmem + kColO, sr.tmem + kColP + 32 + kk * 8, v_desc + (unsigned long long)((kTileBytes + kk * 2048) >> 4), kIdescPV, 1u, two);
                tc_commit(&sc->pv_done);
                tc_commit_if(&sc->o_done, pend_last ? 1u : 0u);
                tc_commit(&sc->empty[g]);
                tile_n += pend_last ? 1u : 0u;
                ++pv_n;
            }
            pend_cnt = cnt;
            pend_fresh = tile_fresh;
            pend_last = false;
            tile_fresh = tile_fresh && cnt == 0u;
            tile_steps = tile_steps || cnt != 0u;
        }
        if (fail) break;
        if (last) {
            tc_commit(&sc->q_empty[qs]);        // every Q K^T of the tile has been issued
            pend_last = tile_steps;             // the tile's last P V is the pending one (the tile's last segment may be empty)
        }
        mbar_arrive(&sc->sched_empty[ss]);
        ++sched_n;
        if (w < 0) break;
    }
    if (fail) give_up(abort_flag, p.status, fail);
}

// ------------------------------------------------------------------------------------------------ softmax (one warpgroup per stream, one thread per row)
__device__ __forceinline__ void softmax_role(const KernelParams& p, SmemCtl* ctl, const StreamRef& sr, int warp, int lane) {
    StreamCtl* sc = sr.sc;
    int* abort_flag = &ctl->abort_flag;
    const int quad = warp & 3;                      // tensor-memory lanes this warp may touch: 32*quad .. +31
    const int row = quad * 32 + lane;               // row of the 128-row tile
    const bool lower = row >= kBlock;
    const int my_who = lower ? kLowerHalf : kUpperHalf;
    const unsigned lane_addr = sr.tmem + ((unsigned)(quad * 32) << 16);
    const float sl2 = p.scale_log2;
    unsigned sched_n = 0, grp_n = 0, msg_n = 0;
    bool ok = true;
    int fail = 0;                                   // code of the wait that was abandoned, if any
    float m_ref = -INFINITY, l_sum = 0.f;
    bool o_dirty = false;                           // has any P V been issued for this tile yet
    // exponentials of the 64 scores of one key block, packed in place: afterwards s[0..31] hold the bit
    // patterns of the 32 words of bf16 probability pairs (four partial sums, so that the adds do not form one chain)
    auto exp_pack = [&](float* s, float neg_m, float& sum0, float& sum1) {
        float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            float x0, x1, p0, p1;
            ffma2(x0, x1, s[2 * j], s[2 * j + 1], sl2, neg_m);
            p0 = ex2(x0);
            p1 = ex2(x1);
            if (j & 1) fadd2(b0, b1, p0, p1);
            else fadd2(a0, a1, p0, p1);
            s[j] = __uint_as_float(pack_bf16(p0, p1));
        }
        fadd2(a0, a1, b0, b1);
        fadd2(sum0, sum1, a0, a1);
    };
    while (ok) {
        const unsigned ss = sched_n % kSchedSlots, sp = (sched_n / kSchedSlots) & 1u;
        if (!mbar_wait(&sc->sched_full[ss], sp, abort_flag)) { fail = 30; break; }
        __syncwarp();
        const WorkSlot* slot = &sc->slot[ss];
        const int w = slot->w, flags = slot->flags, n = slot->n_chunks;
        if (w < 0) {                                // tell the epilogue that this stream is finished
            // (once it has taken the last tile: only then is it known to have read every earlier message, so that
            // the entry reused here is free)
            if (msg_n > 0 && !mbar_wait(&sc->o_free, (msg_n - 1) & 1u, abort_flag)) { fail = 36; break; }
            EpiMsg* msg = &sc->epi[msg_n & 1u];
            if (row == 0) msg->kind = kEpiDone;
            mbar_arrive(&sc->epi_full[msg_n & 1u]);
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
            ok = mbar_wait(&sc->s_full, grp_n & 1u, abort_flag);
            if (!ok) { fail = 31; break; }
            __syncwarp();                           // lanes leave the wait one by one: back in step before the warp-wide loads
            tc_fence_after();
            // A key block with padded keys (rare: the one holding a sequence's end) gets -inf written over their
            // scores in tensor memory first, so that the common path below carries no masking code at all.
            if (__builtin_expect(((who0 | who1) & kHasPadding) != 0, 0)) {
#pragma unroll 1
                for (int c = 0; c < cnt; ++c)
                    if ((c == 0 ? mine0 : mine1) && (e[c].who & kHasPadding)) mask_scores(lane_addr + kColS + 64 * c, e[c].kb);
            }
            float s[128];
            if (mine0) tmem_ld64(lane_addr + kColS, s);
            if (mine1) tmem_ld64(lane_addr + kColS + 64, s + 64);
            tmem_wait_ld();
            // the score columns are free again: the next step's Q K^T may overwrite them
            tc_fence_before();
            mbar_arrive(&sc->s_free);
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
                ok = mbar_wait(&sc->pv_done, (grp_n - 1) & 1u, abort_flag);
                if (!ok) { fail = 32; break; }
                __syncwarp();
                tc_fence_after();
            }
            if (__builtin_expect(rescale && o_dirty, 0)) rescale_accumulator(lane_addr + kColO, alpha);
            if (mine0) tmem_st32(lane_addr + kColP, reinterpret_cast<unsigned*>(s));
            else tmem_st32_zero(lane_addr + kColP);
            if (cnt > 1) {
                if (mine1) tmem_st32(lane_addr + kColP + 32, reinterpret_cast<unsigned*>(s + 64));
                else tmem_st32_zero(lane_addr + kColP + 32);
            }
            if (!ok) break;
            l_sum = l_sum * alpha + (sum0 + sum1);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&sc->p_full);
            ++grp_n;
            o_dirty = true;
        }
        if (!ok) break;
        if (flags & kSegLast) {
            // -------------------------------------------------------- end of the tile: lse now, the output rows via the epilogue
            const int my_q = lower ? slot->qb : slot->qa;
            const unsigned long long qbits = lower ? slot->qbits_b : slot->qbits_a;
            const bool have = live && o_dirty;
            const int part_slot = slot->part_slot;
            const int r64 = row & (kBlock - 1);
            float inv = 0.f;
            if (part_slot >= 0) {
                // one part of a split tile: (max, sum) from here, the raw accumulator from the epilogue
                float* part = p.partials + (size_t)part_slot * kPartialFloats;
                part[128 * 64 + row] = have ? m_ref : -INFINITY;
                part[128 * 64 + 128 + row] = have ? l_sum : 0.f;
            } else if (my_q >= 0) {                 // warp-uniform
                const bool good = have && ((qbits >> r64) & 1ull) && l_sum > 0.f;
                const size_t tok = ((size_t)slot->bh * p.nb + my_q) * kBlock + r64;
                if (p.lse) p.lse[tok] = good ? (m_ref + __log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
                inv = good ? __frcp_rn(l_sum) : 0.f;
                if (!have) {                        // no key block was attended: the row is zeros, written from here
                    uint4* dst = reinterpret_cast<uint4*>(p.out + tok * kBlock);
                    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int j = 0; j < 8; ++j) dst[j] = z;
                }
            }
            if (have) {                             // CTA-uniform per stream: every thread of the warpgroup posts
                EpiMsg* msg = &sc->epi[msg_n & 1u];
                msg->inv[row] = inv;
                if (row == 0) {
                    msg->kind = kEpiTile;
                    msg->bh = slot->bh;
                    msg->qa = slot->qa;
                    msg->qb = slot->qb;
                    msg->part_slot = part_slot;
                }
                mbar_arrive(&sc->epi_full[msg_n & 1u]);      // (release: the message is visible to whoever sees the phase complete)
                ++msg_n;
            }
        }
        tc_fence_before();
        mbar_arrive(&sc->sched_empty[ss]);
        ++sched_n;
    }
    if (fail) give_up(abort_flag, p.status, fail);
}

// ------------------------------------------------------------------------------------------------ epilogue (one warpgroup, both streams)
// Each warp serves its 32 rows of whichever stream has a finished tile: accumulator out of tensor memory,
// scaled by 1/l, to the output rows (or raw, to the scratch of a split tile's part).
__device__ __forceinline__ void epilogue_role(const KernelParams& p, SmemCtl* ctl, unsigned char* smem, unsigned tmem, int warp, int lane) {
    int* abort_flag = &ctl->abort_flag;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int r64 = row & (kBlock - 1);
    const bool lower = row >= kBlock;
    // per stream, packed so that the loop below is one copy of the code: bits 0..15 messages taken, 16..30 tiles
    // taken (only parities are used), bit 31 the stream is finished
    unsigned state0 = 0u, state1 = 0u;              // (scalars: an indexed array would live in local memory)
    IdleClock idle;
    while (!((state0 & state1) >> 31)) {
        bool progress = false;
#pragma unroll 1
        for (int s = 0; s < kStreams; ++s) {
            const unsigned st = s == 0 ? state0 : state1;
            if (st >> 31) continue;
            StreamCtl* sc = &ctl->st[s];
            const unsigned msg_n = st & 0xffffu, tile_n = (st >> 16) & 0x7fffu;
            const unsigned e = msg_n & 1u, eph = (msg_n >> 1) & 1u;
            if (!__all_sync(0xffffffffu, mbar_test(&sc->epi_full[e], eph))) continue;
            progress = true;
            const EpiMsg* msg = &sc->epi[e];
            const unsigned st_next = msg->kind == kEpiDone ? (st | 0x80000000u) : (((msg_n + 1u) & 0xffffu) | (((tile_n + 1u) & 0x7fffu) << 16));
            if (s == 0) state0 = st_next; else state1 = st_next;
            if (st_next >> 31) continue;
            const int bh = msg->bh, my_q = lower ? msg->qb : msg->qa, part_slot = msg->part_slot;
            const float inv = msg->inv[row];
            if (!mbar_wait(&sc->o_done, tile_n & 1u, abort_flag)) { give_up(abort_flag, p.status, 40); return; }
            tc_fence_after();
            const unsigned lane_addr = tmem + s * kStreamCols + ((unsigned)(quad * 32) << 16);
            // the row's destination: the output tensor, or (raw fp32) the scratch of a split tile's part
            const bool partial = part_slot >= 0;
            unsigned char* dst = partial ? reinterpret_cast<unsigned char*>(p.partials + (size_t)part_slot * kPartialFloats + row * 64)
                                         : reinterpret_cast<unsigned char*>(p.out + (((size_t)bh * p.nb + (my_q >= 0 ? my_q : 0)) * kBlock + r64) * kBlock);
            bool write = partial || my_q >= 0;              // warp-uniform
            if (!BB_CHECK(bh >= 0 && bh < p.BH && my_q < p.nb && part_slot < p.BH * max(p.split_tiles_per_head, 1) * p.max_parts, 74)) write = false;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                float o[32];
                tmem_ld32(lane_addr + kColO + c * 32, o);
                tmem_wait_ld();
                if (c == 1) { tc_fence_before(); mbar_arrive(&sc->o_free); }       // the accumulator has been taken
                if (!write) continue;
                if (partial) {
                    float4* d4 = reinterpret_cast<float4*>(dst) + 8 * c;
#pragma unroll
                    for (int j = 0; j < 8; ++j) d4[j] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                } else {
                    uint4* d4 = reinterpret_cast<uint4*>(dst) + 4 * c;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16(o[8 * j + 0] * inv, o[8 * j + 1] * inv);
                        v.y = pack_bf16(o[8 * j + 2] * inv, o[8 * j + 3] * inv);
                        v.z = pack_bf16(o[8 * j + 4] * inv, o[8 * j + 5] * inv);
                        v.w = pack_bf16(o[8 * j + 6] * inv, o[8 * j + 7] * inv);
                        d4[j] = v;
                    }
                }
            }
        }
        if (progress) idle.reset();
        else {
            // (a short sleep, not a suspended wait on one stream's barrier: that would not see the other stream's
            // message for up to 4 us, and the stream's next tile cannot overwrite the accumulator before it is taken)
            __nanosleep(400);
            if (!__all_sync(0xffffffffu, idle.tick(abort_flag, p.status, 41, 0))) return;
        }
    }
}

// ------------------------------------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const KernelParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + kSmemCtl);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStreams; ++s) {
            StreamCtl* sc = &ctl->st[s];
            for (int i = 0; i < kRingGroups; ++i) { mbar_init(&sc->full[i], 1); mbar_init(&sc->empty[i], 1); }
            for (int i = 0; i < 2; ++i) { mbar_init(&sc->q_full[i], 1); mbar_init(&sc->q_empty[i], 1); mbar_init(&sc->epi_full[i], kSoftmaxThreads); }
            mbar_init(&sc->s_full, 1);
            mbar_init(&sc->s_free, kSoftmaxThreads);    // every softmax thread arrives itself: converging the warp and
            mbar_init(&sc->p_full, kSoftmaxThreads);    // electing a lane was measured 10% slower on the whole kernel
            mbar_init(&sc->pv_done, 1);
            mbar_init(&sc->o_done, 1);
            mbar_init(&sc->o_free, kSoftmaxThreads);    // the 128 epilogue threads
            for (int i = 0; i < kSchedSlots; ++i) { mbar_init(&sc->sched_full[i], 1); mbar_init(&sc->sched_empty[i], 3 + kSoftmaxThreads); }    // two producer lanes, the MMA thread, the softmax threads
        }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kWarpProducer) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = *(volatile unsigned*)&ctl->tmem_base;
    const StreamRef s0{&ctl->st[0], smem, tmem};
    const StreamRef s1{&ctl->st[1], smem + kStreamSmemBytes, tmem + kStreamCols};

    if (warp < kWarpEpilogue) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        softmax_role(p, ctl, warp < 4 ? s0 : s1, warp, lane);
    } else if (warp < kWarpProducer) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsEpilogue));
        epilogue_role(p, ctl, smem, tmem, warp, lane);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLight));
        if (warp == kWarpScheduler) scheduler_role(p, ctl, lane);
        else if (warp == kWarpProducer) { if (lane < 2 * kStreams) producer_role(p, ctl, (lane & 1) ? s1 : s0, lane >= kStreams, &tm_q, &tm_k, &tm_v); }
        else if (lane == 0) mma_role(p, ctl, warp == kWarpMma ? s0 : s1);
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
    if (warp == kWarpProducer) {
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
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(&bar, 0u, &abort_flag)) give_up(&abort_flag, status, 99);
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
    wait_expiry_selftest_kernel<<<1, 32, 0, stream>>>(sc.status);
    return cudaGetLastError();
}

namespace {

// Per device, once, with that device current: the kernel's shared-memory attribute (a per-device property of the
// function) and the device's SM count.
struct KernelDevice {
    bool ready = false;
    int sm_count = 0;
};
constexpr int kMaxKernelDevices = 64;
std::mutex g_kernel_mu, g_launch_mu;
KernelDevice g_kernel_dev[kMaxKernelDevices];

cudaError_t kernel_setup(int device, int* sm_count) {
    if (device < 0 || device >= kMaxKernelDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_kernel_mu);
    KernelDevice& d = g_kernel_dev[device];
    if (!d.ready) {
        cudaError_t e = cudaFuncSetAttribute(attn_fwd_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        d.ready = true;
    }
    *sm_count = d.sm_count;
    return cudaSuccess;
}

// One CTA per SM, each running kStreams tile streams.
int grid_size(int sm_count, int total_work) {
    int grid = sm_count;
    const int needed = (total_work + kStreams - 1) / kStreams;
    if (grid > needed) grid = needed;
    return grid < 1 ? 1 : grid;
}

}  // namespace

int launch_attn_fwd_sm100(const FwdArgs& a, const bigbird_layout& L, const DeviceLayout& dl, DeviceScratch& sc,
                          int* launches, cudaError_t* cuda_err) {
    *cuda_err = cudaSuccess;
    if (!(a.scale > 0.f) || !(a.scale < INFINITY)) return BIGBIRD_EINVAL;
    const int64_t rows = (int64_t)a.B * a.H * a.N;
    if (rows >= (1ll << 31) || (int64_t)a.B * a.H * L.items_per_head >= (1ll << 31)) return BIGBIRD_EUNSUPPORTED;

    // One host thread at a time past this point: the per-device scratch bookkeeping below (counter slots, grown
    // buffers) is plain data.
    std::lock_guard<std::mutex> launch_lock(g_launch_mu);
    int device = 0, sm_count = 0;
    cudaError_t de = cudaGetDevice(&device);
    if (de == cudaSuccess) de = kernel_setup(device, &sm_count);
    if (de != cudaSuccess) { *cuda_err = de; return BIGBIRD_ECUDA; }

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

    const int grid = grid_size(sm_count, p.total_work);
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
// and the device copy of the layout's tile schedule, which is sent again whenever another layout is used.
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
    uint64_t schedule_uid = 0;                  // layout whose schedule the array holds (0: none)
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
        int sms = 0;
        e = kernel_setup(device, &sms);
        if (e != cudaSuccess) return e;
        d.sm_count = sms;
        d.base = (unsigned char*)ptr;
    }
    *out = d;
    return cudaSuccess;
}

void static_remember_schedule(int device, uint64_t uid) {
    std::lock_guard<std::mutex> lock(g_static_mu);
    g_static_dev[device].schedule_uid = uid;
}
void static_forget_schedule(int device) { static_remember_schedule(device, 0); }

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
    // The schedule is sent only when the array does not hold this layout's already (copies from the handle's own
    // host arrays, which live as long as the handle).
    if (sd.schedule_uid != L->uid) {
        e = cudaMemcpyAsync(items_dev, L->items_abs.data(), n_items * sizeof(Item), cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess && n_steps) e = cudaMemcpyAsync(steps_dev, L->steps.data(), n_steps * sizeof(Step), cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) { static_forget_schedule(device); return BIGBIRD_ECUDA; }
        static_remember_schedule(device, L->uid);
    }

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
    const int grid = grid_size(sd.sm_count, p.total_work);
    attn_fwd_sm100_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, p);
    if (cudaGetLastError() != cudaSuccess) return BIGBIRD_ECUDA;
    return BIGBIRD_OK;
}

extern "C" int bigbird_last_status_static(void* stream, int* status, int* detail) {
    using namespace bigbird;
    if (!status) return BIGBIRD_EINVAL;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return BIGBIRD_ECUDA;
    if (device < 0 || device >= 64) return BIGBIRD_EUNSUPPORTED;
    StaticDevice sd;
    if (static_setup(device, &sd) != cudaSuccess) return BIGBIRD_ECUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BIGBIRD_ECUDA;
    int host[2] = {0, 0};                       // a stack buffer: nothing is allocated
    if (cudaMemcpy(host, sd.base, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return BIGBIRD_ECUDA;
    *status = host[0];
    if (detail) *detail = host[1];
    return BIGBIRD_OK;
}
