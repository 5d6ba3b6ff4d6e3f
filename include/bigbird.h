/*
 * bigbird.h -- C ABI of the BigBird block-sparse attention forward library for NVIDIA B200 (sm_100a).
 *
 * The operation is the generalised attention of arXiv 2007.14062, Sec. 2, Eq. (AT), restricted to its
 * per-head softmax core:
 *
 *     out[i] = sum_{k in N(i)} softmax_k( scale * q_i . k_k ) v_k ,    lse[i] = ln sum_{k in N(i)} exp(scale * q_i . k_k)
 *
 * where the out-neighbour sets N(i) are those of the block-sparse BigBird graph of App. D: with the
 * sequence cut into blocks of b tokens, query block j attends to the w key blocks of its sliding window
 * (j-(w-1)/2 .. j+(w-1)/2), to the g global blocks and to r random key blocks; global query blocks attend
 * to every block (Sec. 2: A(i,:) = A(:,i) = 1 for i in G).  ITC makes existing blocks global, ETC puts the
 * global tokens in front of the sequence (matrix B of Sec. 2).
 *
 * Conventions
 *   - every function returns BIGBIRD_OK (0) or a negative error code; nothing throws, aborts or traps;
 *   - "host" / "device" in a comment says where the pointer must live;
 *   - the caller owns every buffer it passes; the library owns layout handles until they are destroyed;
 *   - one GPU per call: the device that is current on the calling thread.
 */
#ifndef BIGBIRD_H_
#define BIGBIRD_H_

#include <stdint.h>

#if defined(__GNUC__)
#define BIGBIRD_API __attribute__((visibility("default")))
#else
#define BIGBIRD_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    BIGBIRD_OK = 0,
    BIGBIRD_EINVAL = -1,        /* null pointer, N % b != 0, even w, g > N/b, layout built for another N/b/H ... */
    BIGBIRD_EUNSUPPORTED = -2,  /* shape or dtype outside what the kernels implement */
    BIGBIRD_ECUDA = -3,         /* a CUDA call failed; see bigbird_last_cuda_error() */
    BIGBIRD_ETIMEOUT = -4,      /* a bounded wait inside a kernel expired (reported by bigbird_last_status) */
    BIGBIRD_ENOMEM = -5,
    BIGBIRD_ELIMIT = -6,        /* the problem exceeds the fixed scratch of bigbird_attn_fwd_static */
    BIGBIRD_EINTERNAL = -7      /* a checked build (compiled with BB_DEBUG) found an index out of range inside a kernel; reported by
                                   bigbird_last_status like BIGBIRD_ETIMEOUT, with the code of the check; the kernel skips the access */
};

enum { BIGBIRD_ITC = 0, BIGBIRD_ETC = 1 };
enum { BIGBIRD_FP32 = 0, BIGBIRD_BF16 = 1 };

typedef struct bigbird_layout bigbird_layout;   /* opaque */

/*
 * bigbird_build_layout -- the attention graph of App. D as per-(head, query block) key-block lists.
 *
 *   N     total tokens per sequence (ETC: including the prepended global tokens); N % b == 0
 *   b     block size in tokens
 *   w     sliding-window width in blocks, odd: query block j sees key blocks j-(w-1)/2 .. j+(w-1)/2,
 *         clipped at the ends of the sequence (App. D item 2)
 *   g     number of global blocks (Sec. 2; App. D item 3).  mode BIGBIRD_ITC: the first ceil(g/2) and the last
 *         floor(g/2) blocks; mode BIGBIRD_ETC: the first g blocks
 *   r     random key blocks per (head, non-global query block) (App. D item 1), drawn without replacement
 *         from the ascending list of blocks that are neither in the query block's window nor global (all of
 *         them if fewer than r).  The same for every batch element; not symmetrised (the graph is directed).
 *   seed  selects the random blocks; seed < 2^24, else BIGBIRD_EINVAL (the stream key below gives it 24 bits).
 *         The paper fixes no generator; this library's is: a SplitMix64 stream
 *         with initial state (seed << 40) ^ (h << 20) ^ j for head h and query block j (h, j < 2^20), the
 *         bounded draw floor(z * m / 2^64), and a partial Fisher-Yates shuffle of the candidate list
 *         (for t < r: swap entries t and t + draw(m - t)); the first r entries are taken.
 *   H     number of heads
 *
 * Row (h, j) of the result lists its key blocks in ascending order without duplicates; a global query
 * block lists all N/b blocks.  The handle also carries the device-side schedule derived from the lists;
 * device memory for it is allocated on the first bigbird_attn_fwd that uses the handle.
 * Host-only; thread-safe for distinct handles.  Errors: BIGBIRD_EINVAL, BIGBIRD_ENOMEM.
 */
BIGBIRD_API int bigbird_build_layout(int64_t N, int b, int w, int g, int r, uint64_t seed, int H, int mode,
                         bigbird_layout** out_layout);

/* Number of listed (query block, key block) pairs, summed over heads. */
BIGBIRD_API int bigbird_layout_nnz(const bigbird_layout* layout, int64_t* nnz);

/* Copies the lists out as CSR over rows h * (N/b) + j.  row_ptr: host int32[H * N/b + 1];
 * col_idx: host int32[nnz].  Both caller-owned. */
BIGBIRD_API int bigbird_layout_export(const bigbird_layout* layout, int32_t* row_ptr, int32_t* col_idx);

/* The same graph by key block (what the gradients of K and V walk): row h * (N/b) + c lists, ascending, the query
 * blocks that attend key block c.  col_ptr: host int32[H * N/b + 1]; row_idx: host int32[nnz].  Both caller-owned. */
BIGBIRD_API int bigbird_layout_export_transposed(const bigbird_layout* layout, int32_t* col_ptr, int32_t* row_idx);

/*
 * Introspection of the tile schedule derived from the lists (used by the tests; not needed to run attention).
 * The tensor-core kernel stacks two query blocks into one 2b-row tile (upper half, lower half) and walks a
 * list of steps; a step is one key block together with the halves of the tile that attend it.
 *   sizes   host int32[4]: items per head, leading "heavy" (global-tile) items per head, total steps, heads
 *   items   host int32[H * items_per_head * 8] or NULL: per item (qa, qb, step_begin, step_count, part, nparts, tile, 0),
 *           qa / qb the query blocks of the upper / lower half (qb == -1: none), step_begin relative to the
 *           head's first step
 *   step_base host int32[H] or NULL: first step of each head
 *   steps   host int32[total_steps * 2] or NULL: (key block, who) with who = 0 both halves, 1 upper half only,
 *           2 lower half only
 */
BIGBIRD_API int bigbird_layout_schedule(const bigbird_layout* layout, int32_t* sizes, int32_t* items, int32_t* step_base,
                            int32_t* steps);

/* Frees the handle and the device memory it holds.  No kernel using it may still be running. */
BIGBIRD_API int bigbird_layout_destroy(bigbird_layout* layout);

/*
 * bigbird_attn_fwd -- Eq. (AT) over the graph held by `layout`, for every batch element and head.
 *
 *   q, k, v   device, [B, H, N, D] contiguous, fp32 or bf16 according to `dtype`; 16-byte aligned
 *   layout    from bigbird_build_layout with the same N, b, H
 *   key_padding_mask   device uint8 [B, N], 1 = real token, 0 = padding, or NULL for no padding.  A padded key
 *             gets score -inf before the softmax (the paper is silent on padding; the graph does not depend
 *             on the mask).  A padded QUERY row gets out = 0 and lse = -inf.
 *   out       device, [B, H, N, D], same dtype as q
 *   lse       device fp32 [B, H, N], natural log of the softmax denominator of each row; may be NULL
 *   scale     multiplies q.k before the softmax (Eq. (AT) leaves 1/sqrt(d) out; pass it here)
 *   dtype     BIGBIRD_FP32: fp32 arithmetic on CUDA cores.  BIGBIRD_BF16: tcgen05 tensor-core MMAs with fp32
 *             accumulation in tensor memory, fp32 softmax, bf16 output.
 *   stream    cudaStream_t (NULL = default stream).  The call only enqueues work; it never synchronises.
 *
 * Supported: D == 64 and b == 64 for BIGBIRD_BF16; D in {32, 64, 128} and any b for BIGBIRD_FP32.
 * The first call on a device (and the first call with a larger B, N or a new layout) allocates device
 * scratch owned by the library; later calls allocate nothing.  That scratch (packed mask bits, partial results
 * of split global tiles) is per device: calls that use a key-padding mask or a layout with N/b > 96 must not
 * overlap on the GPU with other such calls (put them on one stream).  Host threads may call concurrently: the
 * library serialises its own bookkeeping.
 * Errors: BIGBIRD_EINVAL, BIGBIRD_EUNSUPPORTED, BIGBIRD_ECUDA, BIGBIRD_ENOMEM.  There is no CPU path.
 */
BIGBIRD_API int bigbird_attn_fwd(const void* q, const void* k, const void* v, const bigbird_layout* layout,
                     const uint8_t* key_padding_mask, void* out, float* lse,
                     int B, int H, int64_t N, int D, int b, float scale, int dtype, void* stream);

/*
 * bigbird_attn_fwd_simt -- the same operation and arguments, always on the CUDA-core kernel (bf16 inputs are
 * widened to fp32 on load).  A slow, independent GPU path kept for debugging the tensor-core kernel.
 */
BIGBIRD_API int bigbird_attn_fwd_simt(const void* q, const void* k, const void* v, const bigbird_layout* layout,
                          const uint8_t* key_padding_mask, void* out, float* lse,
                          int B, int H, int64_t N, int D, int b, float scale, int dtype, void* stream);

/*
 * bigbird_attn_bwd -- gradients of Eq. (AT) over the graph held by `layout` (the paper trains through this
 * operation: Sec. 4 "Pretraining and MLM", App. E.1; it prints no gradient formulas, these are the derivatives of
 * the softmax attention above).  Given dout = d loss / d out:
 *
 *     dv = P^T dout,   dS = P o (dout v^T - rowsum(dout o out)),   dq = scale dS k,   dk = scale dS^T q
 *
 * with P the attention probabilities, recomputed from q, k and the saved lse.
 *
 *   q, k, v, out, dout   device, [B, H, N, D] contiguous, one dtype (fp32 or bf16), 16-byte aligned; out and lse
 *             are the results of bigbird_attn_fwd on the same q, k, v, layout, mask and scale
 *   lse       device fp32 [B, H, N] (required)
 *   dq, dk, dv  device, [B, H, N, D], same dtype; every element is written.  A padded QUERY row gets dq = 0 and gives
 *             nothing to dk, dv; a padded key gets dk = dv = 0.
 * Runs on CUDA cores in fp32 arithmetic for either dtype (D in {32, 64, 128}, any b): a first, correct path; there is
 * no tensor-core gradient kernel yet.  Allocates nothing beyond the layout's device copy; only enqueues work.
 * Errors: BIGBIRD_EINVAL, BIGBIRD_EUNSUPPORTED, BIGBIRD_ECUDA.
 */
BIGBIRD_API int bigbird_attn_bwd(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                     const bigbird_layout* layout, const uint8_t* key_padding_mask, void* dq, void* dk, void* dv,
                     int B, int H, int64_t N, int D, int b, float scale, int dtype, void* stream);

/*
 * bigbird_attn_fwd_static -- bigbird_attn_fwd for callers that must not allocate device memory.  (The paper has
 * no counterpart: this is a property of the library, not of the method.)
 *
 * bigbird_attn_fwd keeps its scratch (status and work-counter words, the packed key-padding bits, the device
 * copy of the layout's schedule) in memory it obtains with cudaMalloc on first use.  Some callers cannot have
 * that: code that runs where device allocation is forbidden or would stall everyone else -- inside a region
 * whose memory is owned by a pool the application sized up front, in a latency-critical serving loop where an
 * implicit device synchronisation is unacceptable, or in a process that has handed all remaining GPU memory to
 * another component.  This entry point calls no cudaMalloc, cudaFree or other allocating routine.  Its scratch
 * is one fixed array of about 1.4 MB that is part of the library image: every GPU that loads the library
 * holds it until the process exits.
 *
 * Arguments, layouts, results and asynchrony are those of bigbird_attn_fwd, with these differences:
 *   - BIGBIRD_BF16 with D == 64 and b == 64 only (the tensor-core kernel); anything else is BIGBIRD_EUNSUPPORTED;
 *   - limits set by the fixed array: B * N/b <= 16384, H * (tiles per head) <= 8192 and at most 131072 schedule
 *     steps summed over heads (bigbird_layout_schedule reports both), and N/b <= 96 (longer sequences have
 *     their global tiles split into parts whose partial results need scratch that grows with B * H); beyond
 *     them the call does nothing and returns BIGBIRD_ELIMIT;
 *   - the array holds the device copy of one layout's schedule.  A call with another layout than the previous
 *     call on that device first copies the new schedule from the handle's host arrays (two cudaMemcpyAsync on
 *     `stream` from pageable memory: the host may wait until they have been staged); later calls with the same
 *     layout enqueue only a 16-byte cudaMemsetAsync and the kernels.  `layout` must not be destroyed while a
 *     call that uses it is being enqueued;
 *   - the first call on a device looks up the array's device address and sets a kernel attribute; make that
 *     first call outside any stream capture;
 *   - all calls on a device share the array, which keeps the contents of the last call: the entry point
 *     re-initialises what must start at zero, but two calls whose kernels overlap on the GPU (different
 *     streams, or different threads) race on it and give undefined results.  Serialise them;
 *   - a bounded wait that expires inside the kernel is reported by bigbird_last_status_static, not by
 *     bigbird_last_status (which reads the allocated scratch of bigbird_attn_fwd); bigbird_last_launch_count and
 *     bigbird_last_cuda_error are not updated.
 * Errors: BIGBIRD_EINVAL, BIGBIRD_EUNSUPPORTED, BIGBIRD_ELIMIT, BIGBIRD_ECUDA.
 */
BIGBIRD_API int bigbird_attn_fwd_static(const void* q, const void* k, const void* v, const bigbird_layout* layout,
                            const uint8_t* key_padding_mask, void* out, float* lse,
                            int B, int H, int64_t N, int D, int b, float scale, int dtype, void* stream);

/*
 * bigbird_last_status_static -- the status of the last bigbird_attn_fwd_static call on the current device:
 * synchronises `stream`, then reads the two status words at the head of the fixed array into a host stack buffer
 * (no allocation).  *status is BIGBIRD_OK or BIGBIRD_ETIMEOUT, *detail (may be NULL) names the wait.  Every
 * bigbird_attn_fwd_static call clears the words when it starts.
 */
BIGBIRD_API int bigbird_last_status_static(void* stream, int* status, int* detail);

/*
 * bigbird_last_status -- synchronises `stream` and reads the device status word of the current device:
 * BIGBIRD_OK, or BIGBIRD_ETIMEOUT if a bounded wait inside a kernel gave up (the kernel then returned early and
 * its outputs are invalid).  *detail (may be NULL) receives a code naming the wait.  Clears the word.
 * The word is one per device, shared by every bigbird_attn_fwd launch on it, so a timeout cannot be attributed to
 * one call among several in flight; after a timeout the function also resets the work counters of every launch
 * slot on that device (with a blocking cudaMemset), which is only safe once all attention kernels on the device
 * have finished.  A debugging facility: call it with the device otherwise idle.
 */
BIGBIRD_API int bigbird_last_status(void* stream, int* status, int* detail);

/*
 * bigbird_selftest_wait_expiry -- failure-detection self-test.  Enqueues a one-thread kernel that waits, with the
 * helper and the limit the attention kernel uses (about two seconds), on a barrier nothing ever signals.  The wait
 * gives up, the kernel returns normally, and the next bigbird_last_status reports BIGBIRD_ETIMEOUT with detail 99;
 * the context stays usable.  Nothing traps, faults or hangs.
 */
BIGBIRD_API int bigbird_selftest_wait_expiry(void* stream);

/* The cudaError_t of the last failed CUDA call made by the library on this thread (0 if none). */
BIGBIRD_API int bigbird_last_cuda_error(void);

/* How many kernels the last bigbird_attn_fwd* call on this thread enqueued. */
BIGBIRD_API int bigbird_last_launch_count(void);

/* A static string for an error code. */
BIGBIRD_API const char* bigbird_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* BIGBIRD_H_ */
