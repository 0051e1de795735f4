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
 * Diagnosis: device address and size of one of the stage's private intermediates after a step
 * (contents of the LAST layer executed).  name is one of
 *   "h"   bf16 [max_tokens, d]      last RMSNorm output
 *   "q"   bf16 [max_tokens, Hq*Dh]  queries after RoPE
 *   "o"   bf16 [max_tokens, Hq*Dh]  attention output
 *   "act" bf16 [max_tokens, F]      silu(gate) * up
 * Errors: INVALID_ARG (unknown name), NO_DEVICE.
 */
hs_status_t hs_stage_debug_buffer(hs_stage_t *stage, const char *name, void **dev_ptr, size_t *bytes);

/*
 * Per-kernel timing of hs_stage_step (measurement support; the paper's analogue is its fixed-SM
 * profiling sweep, Sec. 3.3).  While enabled, every kernel launch of a step is bracketed by CUDA
 * events on the step's stream.  hs_stage_profile_read synchronises those events and adds, per
 * kernel class, the elapsed milliseconds to ms[class] and the launch count to launches[class]
 * (host arrays of HS_PROFILE_CLASSES entries, accumulated since the last read), then forgets them.
 * Classes: 0 rmsnorm, 1 qkv gemm, 2 prefill attention, 3 decode attention, 4 decode combine,
 * 5 out-proj gemm, 6 gate/up gemm, 7 down gemm.
 * Errors: INVALID_ARG, NO_DEVICE, CUDA.
 */
#define HS_PROFILE_CLASSES 8
hs_status_t hs_stage_profile_enable(hs_stage_t *stage, int32_t enable);
hs_status_t hs_stage_profile_read(hs_stage_t *stage, float *ms, int32_t *launches);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HORIZONSERVE_OPS_H_ */
