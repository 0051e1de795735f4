/*
 * horizonserve_ops.h -- kernel-level entry points of the library: the building blocks of
 * hs_stage_step exposed on their own for unit parity tests, micro-benchmarks and diagnosis.
 * Same conventions as horizonserve.h (device pointers are borrowed, calls enqueue on the given
 * stream and return without synchronising, no call allocates device memory).
 */
#ifndef HORIZONSERVE_OPS_H_
#define HORIZONSERVE_OPS_H_

#include "horizonserve.h"

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default) /* the declarations below are the library's exported surface */
#endif

/*
 * The dense contraction of the step (the projections of the decoder layer; the paper prints no
 * formula for them): out[M,N] (fp32) = a[M,K] (bf16, row-major) * w[N,K]^T (bf16, row-major, i.e.
 * [out_features, in_features]) + resid[M,N] (fp32, nullable, may alias out; when it is a different buffer it
 * is first copied to out, and the product is then added in place), fp32 accumulation,
 * run as at most sm_budget persistent blocks.  K and N must be multiples of 8; a, w 16-byte aligned.
 * `status_dev` is a device int (zero on entry) that receives HS_ERR_TIMEOUT if a bounded wait inside
 * the kernel runs out; it may not be NULL.
 * Errors: INVALID_ARG, INVALID_BUDGET, UNSUPPORTED_SHAPE, CUDA.
 */
hs_status_t hs_op_gemm_bf16(const void *a, const void *w, const float *resid, float *out, int32_t M, int32_t N,
                            int32_t K, int32_t sm_budget, int32_t *status_dev, void *cuda_stream);

/*
 * The same contraction with `a` and `w` both holding fp16 (IEEE half) values: the form the stage uses by
 * default, its private activations in fp16 (an 11-bit significand) against fp16 copies of the weights.
 */
hs_status_t hs_op_gemm_f16(const void *a, const void *w, const float *resid, float *out, int32_t M, int32_t N,
                           int32_t K, int32_t sm_budget, int32_t *status_dev, void *cuda_stream);

/*
 * Diagnosis: device address and size of one of the stage's private intermediates after a step
 * (contents of the LAST layer executed).  name is one of
 *   "h"   [max_tokens, d]      last RMSNorm output            (fp16; bf16 with HS_FLAG_BF16_ACTIVATIONS).  Where
 *                              the norm is folded into the GEMMs around it (all projections on SM pairs, or a
 *                              step of at most 16 rows; unconditioned stage) this is 16-bit(x o g), not yet scaled
 *                              by the row's rsqrt(mean(x^2) + eps): the GEMM behind it applies that factor.
 *   "q"   [max_tokens, Hq*Dh]  queries after RoPE             (bf16)
 *   "o"   [max_tokens, Hq*Dh]  attention output               (fp16; bf16 with the flag)
 *   "act" [max_tokens, F]      silu(gate) * up                (fp16; bf16 with the flag)
 *   "smid" int32 [8 classes][160]   SM census: asking for this buffer switches the census on for the
 *                                   following steps; entry [class][b] is then 1 + the SM on which block b
 *                                   of the last layer's launch of that kernel class ran (0 = no such
 *                                   block).  Classes as in hs_stage_profile_read.  It shows that a step
 *                                   with sm_budget B never occupies more than B SMs at a time.
 * Errors: INVALID_ARG (unknown name), NO_DEVICE.
 */
hs_status_t hs_stage_debug_buffer(hs_stage_t *stage, const char *name, void **dev_ptr, size_t *bytes);

/*
 * Per-kernel timing of hs_stage_step (measurement support; the paper's analogue is its fixed-SM
 * profiling sweep, Sec. 3.3).  While enabled, every kernel launch of a step is bracketed by CUDA
 * events on the step's stream.  hs_stage_profile_read synchronises those events and adds, per
 * kernel class, the elapsed milliseconds to ms[class] and the launch count to launches[class]
 * (host arrays of HS_PROFILE_CLASSES entries, accumulated since the last read), then forgets them.
 * While enabled, the kernels of a step never overlap (the events between them serialise the stream; the prefill
 * and decode attention kernels of a layer, which otherwise run side by side on two shares of the budget, run one
 * after the other on the whole budget), so the per-class times add up to more than an unprofiled step takes.
 * A residual GEMM that folds the RMSNorm behind it is timed with that work (classes 5 and 7); class 0 then counts
 * the one norm launch a step keeps.
 * Classes: 0 rmsnorm, 1 qkv gemm, 2 prefill attention, 3 decode attention (with the merge of its split
 * partials), 4 unused (always zero; kept so that the class numbers stay what they were),
 * 5 out-proj gemm, 6 gate/up gemm, 7 down gemm.
 * Errors: INVALID_ARG, NO_DEVICE, CUDA.
 */
#define HS_PROFILE_CLASSES 8
hs_status_t hs_stage_profile_enable(hs_stage_t *stage, int32_t enable);
hs_status_t hs_stage_profile_read(hs_stage_t *stage, float *ms, int32_t *launches);

/*
 * Diagnosis of the bounded waits (the paper has no counterpart; it concerns this library's kernels only).  Every
 * wait inside the step's kernels gives up after a time limit, records HS_ERR_TIMEOUT in the device status word
 * and lets its block wind down in order -- roles leave their loops, copies in flight are given time to land,
 * tensor memory is freed -- so a lost signal ends as an error code, never as a hung GPU.  This call runs that
 * sequence on purpose: one small block waits on a barrier that nobody signals, with the caller's limit
 * (limit_ns nanoseconds, 1 us .. 100 ms) in place of the kernels' 2 s.  After the stream has been synchronised
 * *status_dev (a device int, zero on entry) holds HS_ERR_TIMEOUT and *waited_ns_dev (device uint64, nullable) the
 * time the first waiter spent; the context remains usable.
 * Errors: INVALID_ARG (NULL status, limit out of range), CUDA.
 */
hs_status_t hs_op_wait_probe(uint64_t limit_ns, int32_t *status_dev, uint64_t *waited_ns_dev, void *cuda_stream);

/*
 * Decode attention for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this call: it is a packaging variant of the decode-attention kernel of hs_stage_step.)
 *
 * Who needs it: a process that gave all free HBM to its KV pool at start-up, or a component that only
 * receives device pointers from its host runtime, cannot provide the scratch workspace that the stage
 * API expects -- an allocation at that point fails or stalls every stream of the GPU.  Here the
 * scratch (split-KV partials, work-queue head, the call's integer metadata, about 4.3 MB) is a fixed
 * array inside the library image; every GPU that loads the library carries it until the process
 * ends.  The call itself calls no allocating routine: no cudaMalloc, cudaFree or cudaHostAlloc, no heap, and no
 * library that allocates; its host-side metadata lives in a fixed array of the library image.
 *
 * Computes, for each of n_seqs sequences, o[s] = softmax(q[s] K^T / sqrt(head_dim)) V over keys
 * 0 .. kv_len[s]-1 of that sequence (grouped-query: query head h reads KV head h / (n_q_heads /
 * n_kv_heads)), exactly as the decode part of hs_stage_step does.
 *   q_dev, o_dev   device bf16 [n_seqs, n_q_heads * head_dim], 16-byte aligned; q is used as given
 *                  (apply RoPE before); o is overwritten.
 *   kv_pool_dev    device bf16 pool in the layout of hs_kv_pool_bytes, 256-byte aligned; `layer`
 *                  selects the layer, n_layers / num_pages describe the pool.
 *   kv_len         host [n_seqs], >= 1; block_tables: host [n_seqs * max_pages_per_seq].
 * Limits (the size of the fixed scratch): n_seqs <= HS_NOALLOC_MAX_SEQS, max_pages_per_seq <=
 * HS_NOALLOC_MAX_PAGES_PER_SEQ, and sum over sequences of n_kv_heads * ceil(kv_len / 256) <=
 * HS_NOALLOC_MAX_ITEMS; anything larger is refused with HS_ERR_UNSUPPORTED_SHAPE and nothing runs.
 * The first call on a device resolves the scratch array's device address and configures the kernels;
 * make that first call before any stream capture begins.  All calls share the one scratch area: it
 * keeps the previous call's contents, the parts that must start from zero are cleared by each call,
 * and two calls whose kernels can overlap on the GPU (different streams, no ordering between them)
 * race on it -- order them.  The work is enqueued on cuda_stream.  The metadata travels by an asynchronous copy
 * from ordinary (pageable) host memory, so the call may wait on the host until earlier work of that stream has
 * finished; it does not wait for its own kernel.  Calls from several host threads are serialised inside.
 * If a bounded wait inside the kernel runs out, the kernel ends in order and records HS_ERR_TIMEOUT in a status
 * word of the scratch area; hs_op_decode_attention_noalloc_status (after synchronising the stream) copies the
 * status word of the most recent call to *status_out (HS_OK = 0 when nothing went wrong).
 * Errors: INVALID_ARG, INVALID_BUDGET, UNSUPPORTED_SHAPE, BAD_BLOCK_TABLE, CUDA.
 */
#define HS_NOALLOC_MAX_SEQS 64
#define HS_NOALLOC_MAX_PAGES_PER_SEQ 256
#define HS_NOALLOC_MAX_ITEMS 512
hs_status_t hs_op_decode_attention_noalloc(const void *q_dev, const void *kv_pool_dev, int32_t n_layers, int32_t layer,
                                           int32_t num_pages, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                           int32_t n_seqs, const int32_t *kv_len, const int32_t *block_tables,
                                           int32_t max_pages_per_seq, void *o_dev, int32_t sm_budget,
                                           void *cuda_stream);
hs_status_t hs_op_decode_attention_noalloc_status(int32_t *status_out);

/*
 * Host-only diagnosis of the planner: the attention work lists hs_stage_step would build for `batch` (validated as
 * by hs_stage_plan; works on a stage without a device, which plans for 148 SMs).  The paper has no counterpart: it
 * leaves the execution of a step to its runtime (Sec. 5).
 *   decode_items   [decode_cap][8] int32, in the order the kernel's queue hands them out:
 *                  {decode row, KV head, first key, end key (exclusive), sequence, token row, the group's first
 *                  partial slot, items of the group | index within the group << 16}; in group mode (*decode_group = 1:
 *                  a small batch, every (sequence, KV head) group worked by one block) eight page slices per group,
 *                  group-major, some possibly empty (first key = end key), the last two words unused.
 *   prefill_items  [prefill_cap][8] int32, longest first: {sequence, KV head, first new token, tokens (at most two Q
 *                  tiles), cached tokens, token row of the sequence's first new token, new tokens of the sequence, 0}.
 * Any pointer may be NULL; counts are always written when their pointer is given; at most cap records are copied.
 * Errors: INVALID_ARG, BAD_BLOCK_TABLE.
 */
hs_status_t hs_stage_plan_attention(hs_stage_t *stage, const hs_batch_t *batch, int32_t *decode_items, int32_t decode_cap,
                                    int32_t *n_decode_items, int32_t *decode_group, int32_t *prefill_items,
                                    int32_t prefill_cap, int32_t *n_prefill_items);

/*
 * Host-only: the K block (of 64) at which split i (0 .. ks; i = ks gives k_blocks) of a small step's residual GEMM
 * begins when its k_blocks are cut into ks splits.  Each split is ten K blocks longer than the one before it (the
 * splits add their sums one after the other, and a link of that chain takes about as long as ten K blocks take to
 * stream), or all are equal when K is too short for that.  Returns -1 for ks < 1, k_blocks < 1 or i outside 0 .. ks.
 */
int32_t hs_op_gemm_split_begin(int32_t k_blocks, int32_t ks, int32_t i);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HORIZONSERVE_OPS_H_ */
