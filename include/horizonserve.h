/*
 * horizonserve.h -- C ABI of the SM-budgeted shared-stage transformer step.
 *
 * Vocabulary follows the paper: a *stage* is one component of an omni-model
 * pipeline (the shared backbone, or a downstream generator such as a talker;
 * Sec. 2.2); one scheduling step runs a batch on a stage under a per-stage SM
 * cap (Algorithm 1, step 4: "run the batch with cap s_shared"), and the two
 * stages' caps are complementary, s_down = S_tot - s_shared (Sec. 4.3, Eq. 1
 * and the headroom rule after it).  The paper applies the cap with one CUDA
 * context per SM level and notes that any backend exposing a per-stage SM cap
 * will do (Sec. 5); here the cap is the `sm_budget` argument of
 * hs_stage_step: every kernel of the step runs as at most `sm_budget`
 * persistent thread blocks, one per SM, so two stages stepped on two streams
 * with complementary budgets occupy disjoint SMs.
 *
 * What a step computes (the paper keeps its runtime's model execution
 * unchanged and prints no formula; this is the textbook pre-norm decoder
 * layer, "prefill builds the KV cache, decode re-reads weights and the
 * accumulated cache", Sec. 2.1), for each of n_layers layers:
 *     h = rmsnorm(x, g_attn);  q,k,v = h Wq^T, h Wk^T, h Wv^T;  rotate-half
 *     RoPE on q and k at the token's absolute position;  k, v stored as bf16
 *     in the paged cache;  o = causal GQA attention of q over cache positions
 *     0..p (query head hq reads KV head hq / (Hq/Hkv));  x += o Wo^T;
 *     h2 = rmsnorm(x, g_mlp);  x += (silu(h2 Wg^T) * (h2 Wu^T)) Wd^T.
 * Numeric contract: everything that crosses this interface is bf16 storage
 * (x_in, weights, the KV cache) except the fp32 output; accumulation is fp32
 * and the residual stream is fp32.  Inside a step q, K, V and the softmax
 * weights are bf16; the activations that are multiplied with the weights (h,
 * the attention output, the SwiGLU activation) are private to the stage and
 * are held in fp16 (11 significand bits, clamped to +-65504) and multiplied
 * with fp16 copies of the weights that hs_stage_create makes in the workspace
 * (one MMA cannot mix fp16 with bf16; a bf16 weight is an fp16 value exactly
 * when 2^-17 <= |w| <= 65504, smaller ones move by at most 2^-25), which
 * keeps a multi-layer step within the 2e-2 RMS tolerance.
 * HS_FLAG_BF16_ACTIVATIONS keeps those activations in bf16 and reads the
 * caller's bf16 weights directly: no copies, a smaller workspace, the 8-bit
 * significand's larger error.  Every
 * conversion rounds to nearest even; inputs must be finite.  Outputs and the
 * bytes written to the KV cache are bit-identical for every valid sm_budget.
 *
 * Conventions
 *  - No call allocates device memory: the caller (PyTorch in this repository)
 *    owns weights, KV pool, workspace, inputs and outputs and lends the
 *    pointers for the stage's lifetime.  "device" pointers are CUDA device
 *    pointers of the stage's device; "host" pointers are ordinary memory.
 *  - hs_stage_step validates on the host, enqueues on the given stream and
 *    returns without synchronising.  Host-detectable errors are returned
 *    synchronously and nothing is launched.  Anomalies seen on the device
 *    (an exhausted bounded wait) set a status word; the kernels always run
 *    to completion without trapping, and hs_stage_status reports it after
 *    the stream has been synchronised.
 *  - A stage is driven from one host thread and one stream at a time; two
 *    different stages may be stepped concurrently on two streams.
 *  - No function throws; every function that can fail returns hs_status_t.
 */
#ifndef HORIZONSERVE_H_
#define HORIZONSERVE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default) /* the declarations below are the library's exported surface */
#endif

#define HS_ABI_VERSION 1u
#define HS_PAGE_SIZE 16 /* tokens per KV page; the only supported value */
/* Stage flag: keep the private activations that feed the projections (h, attention output o, SwiGLU
 * activation act) in bf16 instead of the default fp16, and make no fp16 copies of the weights -- see the
 * numeric contract above. */
#define HS_FLAG_BF16_ACTIVATIONS 1u
/*
 * No causal mask: every token of a sequence attends to all of the sequence's keys, the cached ones and all new
 * ones of the step (K/V of the whole step are written before any attention runs).  This is the attention of a
 * denoising (DiT-style) block, the kind of downstream visual generator the paper co-locates with the shared stage
 * (Sec. 2.1, Sec. 3.1); such a stage normally runs every step with ctx_len = 0 and frees nothing in between.
 */
#define HS_FLAG_BIDIRECTIONAL 2u

typedef struct hs_stage hs_stage_t; /* opaque; owned by the library */

typedef enum {
  HS_OK = 0,
  HS_ERR_INVALID_ARG = 1,       /* NULL pointer, inconsistent counts, bad ABI version          */
  HS_ERR_INVALID_BUDGET = 2,    /* sm_budget outside [1, SM count of the device]               */
  HS_ERR_UNSUPPORTED_SHAPE = 3, /* head_dim not 64/128, Hq % Hkv != 0, misaligned widths       */
  HS_ERR_OUT_OF_PAGES = 4,      /* hs_kv_alloc: pool exhausted (nothing was allocated)         */
  HS_ERR_BAD_BLOCK_TABLE = 5,   /* page id out of range, too few pages, page shared by two seqs */
  HS_ERR_CUDA = 6,              /* a CUDA runtime/driver call failed                           */
  HS_ERR_TIMEOUT = 7,           /* a bounded wait inside a kernel ran out                      */
  HS_ERR_NO_DEVICE = 8,         /* the stage was created host-only (device = -1)               */
  HS_ERR_UNKNOWN_SEQ = 9        /* hs_kv_free on a sequence that owns no pages                 */
} hs_status_t;

/* Stage description (Sec. 2.2: shared stage / downstream stage).  POD, copied at create. */
typedef struct {
  uint32_t abi_version;      /* HS_ABI_VERSION */
  int32_t device;            /* CUDA ordinal, or -1: host-only stage (allocator + planning, no step) */
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn;
  float rms_eps, rope_base;
  int32_t page_size;         /* must be HS_PAGE_SIZE */
  int32_t num_pages;         /* pages in the KV pool (shared by all layers: page id p is page p of every layer) */
  int32_t max_tokens;        /* most new tokens in one step */
  int32_t max_seqs;          /* most sequences in one step */
  int32_t max_pages_per_seq; /* row length of block tables */
  int32_t max_position;      /* ctx_len + q_len never exceeds this (sizes the RoPE table) */
  uint32_t flags;            /* 0, or an OR of HS_FLAG_BF16_ACTIVATIONS, HS_FLAG_BIDIRECTIONAL */
} hs_stage_config_t;

/* One layer's weights: device pointers to bf16, row-major [out_features, in_features] (biases: hs_stage_set_qkv_bias). */
typedef struct {
  const void *g_attn; /* [d]          gain of the attention RMSNorm */
  const void *w_q;    /* [Hq*Dh, d]   */
  const void *w_k;    /* [Hkv*Dh, d]  */
  const void *w_v;    /* [Hkv*Dh, d]  */
  const void *w_o;    /* [d, Hq*Dh]   */
  const void *g_mlp;  /* [d]          gain of the MLP RMSNorm */
  const void *w_gate; /* [F, d]       */
  const void *w_up;   /* [F, d]       */
  const void *w_down; /* [d, F]       */
} hs_layer_weights_t;

/* One step's batch ("batch B" of Algorithm 1).  Host arrays are consumed before the call returns. */
typedef struct {
  int32_t n_seqs;
  int32_t n_tokens;            /* = sum of q_len */
  const int32_t *q_len;        /* host [n_seqs]: new tokens of each sequence this step (>= 1; 1 = decode) */
  const int32_t *ctx_len;      /* host [n_seqs]: tokens already in the cache; new token j sits at position ctx_len + j */
  const int32_t *block_tables; /* host [n_seqs * max_pages_per_seq]: physical page of each logical page, unused = -1 */
  const void *x_in;            /* device bf16 [n_tokens, d]: input hidden states, sequences concatenated */
  void *y_out;                 /* device fp32 [n_tokens, d]: residual stream after the last layer */
} hs_batch_t;

/*
 * Sizes of the two caller-provided device buffers.
 *  KV pool: bf16 [n_layers][2 (K,V)][num_pages][n_kv_heads][16][head_dim]; K is stored after RoPE.
 *           One (page, head) block is 16*head_dim*2 contiguous bytes.  Must be 256-byte aligned (what cudaMalloc gives).
 *  Workspace: private scratch of the stage (activations, RoPE table, step metadata, attention
 *           partials and, unless HS_FLAG_BF16_ACTIVATIONS is set, fp16 copies of all projection weights, i.e.
 *           as many bytes again as those weights).  Must be 256-byte aligned (what cudaMalloc gives).  Its
 *           contents are meaningless to the caller.
 * Both return 0 for an invalid configuration.
 */
size_t hs_kv_pool_bytes(const hs_stage_config_t *cfg);
size_t hs_workspace_bytes(const hs_stage_config_t *cfg);

/*
 * Creates a stage.  `layers` is a host array of n_layers entries whose members are device pointers;
 * kv_pool_dev and workspace_dev are device buffers of at least the sizes above.  All of them stay
 * owned by the caller and must outlive the stage.  With cfg->device == -1 every device pointer may be
 * NULL and the stage supports only hs_kv_alloc / hs_kv_free / hs_stage_plan.
 * The call reads the weights on the device's default stream (it makes the fp16 copies there) and
 * synchronises the device once, so the weights must be complete when it is made; the stage does not see
 * later changes to them unless HS_FLAG_BF16_ACTIVATIONS is set.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE, CUDA.
 */
hs_status_t hs_stage_create(const hs_stage_config_t *cfg, const hs_layer_weights_t *layers, void *kv_pool_dev,
                            void *workspace_dev, hs_stage_t **out);

/*
 * Page allocator of the stage's KV pool (the paper keeps its runtime's KV management, Sec. 5; the
 * rule here is fixed so that block tables are reproducible).  The free list is a stack whose pops on a
 * fresh pool yield pages 0, 1, 2, ...  hs_kv_alloc grows sequence seq_id to hold total_tokens tokens by
 * popping ceil(total_tokens / 16) - owned pages, then writes the sequence's whole block table to
 * block_table_out (host, `cap` entries; entries past the table are left untouched) and its length to
 * n_pages_out.  On OUT_OF_PAGES or when cap is too small (INVALID_ARG) nothing changes.
 * hs_kv_free returns the sequence's pages in reverse order of acquisition.
 */
hs_status_t hs_kv_alloc(hs_stage_t *stage, int64_t seq_id, int32_t total_tokens, int32_t *block_table_out,
                        int32_t cap, int32_t *n_pages_out);
hs_status_t hs_kv_free(hs_stage_t *stage, int64_t seq_id);
int32_t hs_kv_free_pages(const hs_stage_t *stage); /* pages currently on the free list */

/*
 * Host-only: validates a batch exactly as hs_stage_step does and writes the per-token metadata the
 * kernels will use: owning sequence, absolute position, and cache slot = page * 16 + position % 16
 * (host arrays of n_tokens entries; any may be NULL).  x_in / y_out are not examined.
 * Errors: INVALID_ARG, BAD_BLOCK_TABLE.
 */
hs_status_t hs_stage_plan(hs_stage_t *stage, const hs_batch_t *batch, int32_t *tok_seq, int32_t *tok_pos,
                          int32_t *tok_slot);

/*
 * Runs one step of the stage on `batch` using at most sm_budget SMs, enqueued on cuda_stream (a
 * cudaStream_t; NULL = the default stream).  For each sequence the q_len new tokens occupy positions
 * ctx_len .. ctx_len + q_len - 1; their K/V are written to the cache pages named by the block table and
 * every new token attends causally to positions 0..p.  y_out receives all n_tokens rows.  Re-running
 * the same step rewrites the same slots with the same values.  The caller advances ctx_len itself.
 * With sm_budget < the device's SM count every kernel of the step starts only after the previous one has
 * ended, so that no block of the step ever sits on an SM outside the budget; with sm_budget == SM count
 * (no co-running neighbour) each kernel's set-up overlaps the previous kernel's drain.  A decode-only step of at
 * most 16 rows under a partial budget runs, after its first RMSNorm, as one cooperative launch of at most sm_budget
 * blocks whose phases are the same kernels' bodies separated by bounded grid-wide barriers (same results; the
 * separate launches are used instead where the device refuses a cooperative launch).  With both prefill and decode
 * work in a step the two attention kernels of a layer run side by side on two shares of the budget, the decode
 * kernel on a stream of the stage's own that is forked from and joined to cuda_stream by events.
 * Errors (nothing launched): INVALID_ARG, INVALID_BUDGET, BAD_BLOCK_TABLE, NO_DEVICE, CUDA.
 */
hs_status_t hs_stage_step(hs_stage_t *stage, const hs_batch_t *batch, int32_t sm_budget, void *cuda_stream);

/*
 * Optional biases of one layer's q, k, v projections: q, k, v = h W^T + b, added before RoPE (the paper runs its
 * backbones' model code unchanged, Sec. 5; the 7B-class backbones it serves carry these three biases).
 *   b_q  device bf16 [n_q_heads * head_dim];  b_k, b_v  device bf16 [n_kv_heads * head_dim]
 * 16-byte aligned, borrowed until the stage is destroyed or the layer's biases are set again; any of the three
 * may be NULL (no bias on that projection; the state of a new stage).  Takes effect for steps enqueued after
 * the call.  Errors: INVALID_ARG (NULL stage, layer out of range, misaligned pointer), NO_DEVICE.
 */
hs_status_t hs_stage_set_qkv_bias(hs_stage_t *stage, int32_t layer, const void *b_q, const void *b_k, const void *b_v);

/*
 * Optional per-sequence modulation of a conditioned block (the adaLN-Zero block of diffusion transformers, with
 * this stage's RMSNorm; the paper names such generators as downstream stages, Sec. 2.1, and gives no arithmetic).
 *   mod  device fp32 [n_layers][max_seqs][6][d_model], 16-byte aligned, borrowed until replaced or the stage is
 *        destroyed; NULL switches the modulation off (the state of a new stage).
 * Rows 0..5 of (layer, sequence s) are shift_a, scale_a, gate_a, shift_m, scale_m, gate_m, and the layer computes
 *   h_a = rmsnorm(x) g_attn (1 + scale_a) + shift_a,   x += gate_a * (attention output W_o^T),
 *   h_m = rmsnorm(x) g_mlp  (1 + scale_m) + shift_m,   x += gate_m * (MLP output),
 * element-wise over d_model, where s is the index of the token's sequence in the step's batch.  The vectors are
 * read when a step runs, so they may be rewritten between steps (a new timestep) without another call.
 * Errors: INVALID_ARG (NULL stage, misaligned pointer), NO_DEVICE.
 */
hs_status_t hs_stage_set_modulation(hs_stage_t *stage, const void *mod);

/* Device-side status of the steps run so far (HS_OK or HS_ERR_TIMEOUT); call after synchronising the stream. */
hs_status_t hs_stage_status(hs_stage_t *stage);

/*
 * Saturation report of the stage's private fp16 activations.  h, the attention output and the SwiGLU activation
 * are clamped to +-65504 when they are stored (numeric contract above); *count receives how many stored values
 * were clamped since the stage was created -- 0 for every well-scaled model, and a signal that the step's output
 * is no longer within tolerance otherwise (rerun the stage with HS_FLAG_BF16_ACTIVATIONS, whose range is that of
 * fp32).  Always 0 with that flag.  Call after synchronising the stream.
 * Errors: INVALID_ARG, NO_DEVICE, CUDA.
 */
hs_status_t hs_stage_saturation_count(hs_stage_t *stage, int64_t *count);

/* SM count of the stage's device (S_tot of Eq. 1); 0 for a host-only stage. */
int32_t hs_stage_sm_count(const hs_stage_t *stage);

hs_status_t hs_stage_destroy(hs_stage_t *stage);
const char *hs_status_str(hs_status_t status);

/* Text of the CUDA error behind the calling thread's most recent HS_ERR_CUDA ("" if there was none).
 * The string is owned by the library and valid until the thread's next failing call. */
const char *hs_last_error(void);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HORIZONSERVE_H_ */
