/*
 * horizonserve_head.h -- the two ends of a stage around hs_stage_step: the token embedding in front of it and,
 * behind it, the final RMSNorm, the vocabulary projection and greedy sampling on chosen rows (normally the
 * last token of each sequence).  The paper keeps its runtime's model execution unchanged (Sec. 5) and prints
 * no formula for these; they are the textbook definitions:
 *     x[t, :]      = E[token[t], :]
 *     h[r, :]      = y[row[r], :] * rsqrt(mean(y[row[r], :]^2) + eps) * g_final        (rounded to bf16)
 *     logits[r, v] = sum_i h[r, i] * W_vocab[v, i]                                     (fp32 accumulation)
 *     token[r]     = the lowest v that attains max_v logits[r, v]
 * Same conventions as horizonserve.h: device pointers are borrowed, every call enqueues on the given stream
 * and returns without synchronising, no call allocates device memory, and every kernel runs as at most
 * sm_budget blocks of one per SM, so the calls can share the GPU with another stage like hs_stage_step does.
 * Results do not depend on sm_budget.
 */
#ifndef HORIZONSERVE_HEAD_H_
#define HORIZONSERVE_HEAD_H_

#include "horizonserve.h"

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

typedef struct hs_head hs_head_t; /* opaque, owned by the library */

typedef struct {
  uint32_t abi_version; /* HS_ABI_VERSION */
  int32_t device;       /* CUDA ordinal */
  int32_t d_model;      /* multiple of 8 */
  int32_t vocab;        /* rows of the embedding table and of W_vocab, multiple of 8 */
  float rms_eps;
  int32_t max_rows;     /* most rows sampled by one hs_head_step, 1 .. 128 */
} hs_head_config_t;

/* Bytes of the caller-provided device workspace (256-byte aligned); 0 for an invalid configuration. */
size_t hs_head_workspace_bytes(const hs_head_config_t *cfg);

/*
 * Creates the sampling head.  g_final: device bf16 [d_model]; w_vocab: device bf16 [vocab, d_model], row-major
 * (both 16-byte aligned, borrowed for the head's lifetime).  Errors: INVALID_ARG, UNSUPPORTED_SHAPE, CUDA.
 */
hs_status_t hs_head_create(const hs_head_config_t *cfg, const void *g_final, const void *w_vocab, void *workspace_dev,
                           hs_head_t **out);

/*
 * Samples one token for each of n rows of y.
 *   y       device fp32 [*, d_model]: the y_out of a step
 *   rows    device int32 [n]: which rows of y to sample from (each in range of y; not checked)
 *   logits  device fp32 [n, vocab], 16-byte aligned: receives the logits
 *   tokens  device int32 [n]: receives the sampled token ids
 * Errors (nothing launched): INVALID_ARG (NULL, n outside 1 .. max_rows), INVALID_BUDGET, CUDA.
 */
hs_status_t hs_head_step(hs_head_t *head, const float *y, const int32_t *rows, int32_t n, float *logits,
                         int32_t *tokens, int32_t sm_budget, void *cuda_stream);

/* Device-side status of the calls so far (HS_OK or HS_ERR_TIMEOUT); call after synchronising the stream. */
hs_status_t hs_head_status(hs_head_t *head);

hs_status_t hs_head_destroy(hs_head_t *head);

/*
 * Embedding lookup: x_out[t, :] = table[tokens[t], :] for n tokens.
 *   tokens  device int32 [n];  table: device bf16 [vocab, d_model];  x_out: device bf16 [n, d_model]
 *   (table and x_out 16-byte aligned, d_model a multiple of 8).
 * A token id outside 0 .. vocab-1 yields a row of zeros and sets *status_dev (device int, zero on entry, may
 * not be NULL) to HS_ERR_INVALID_ARG.
 * Errors (nothing launched): INVALID_ARG, INVALID_BUDGET, UNSUPPORTED_SHAPE, CUDA.
 */
hs_status_t hs_op_embed(const int32_t *tokens, int32_t n, const void *table, int32_t vocab, int32_t d_model,
                        void *x_out, int32_t sm_budget, int32_t *status_dev, void *cuda_stream);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HORIZONSERVE_HEAD_H_ */
