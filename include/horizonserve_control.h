/*
 * horizonserve_control.h -- the two host-side controllers around hs_stage_step.  First the spatial one, which
 * chooses the step's sm_budget: the
 * bandwidth-guided SM throttling of the paper (Sec. 4.3, Eq. 1; Algorithm 1 step 3), and the offline choice
 * of the co-running cap from a fixed-SM sweep (Sec. 4.1, "SLO and SM-ladder construction").  Host-only: no
 * call touches a GPU or allocates device memory; all pointers are host pointers.
 *
 * Per step the controller is given A, whether a downstream stage is active, and B, a sample of the
 * memory-bandwidth pressure (any non-negative number whose saturation value is b_sat: the paper samples the
 * NVML memory-activity counter; this repository divides the bytes a tick must move by the tick's duration and
 * by the measured copy bandwidth).  It keeps
 *     Bhat <- gamma * B + (1 - gamma) * Bhat          (exponentially weighted moving average; the first
 *                                                     sample initialises Bhat = B)
 *     rho   = min(max(Bhat / b_sat, 0), 1)
 *     s*    = s_aggr                                                   if A == 0
 *           = snap(ladder, S_min + rho * (S_cap - S_min))              if A != 0          (Eq. 1)
 * where ladder[0] = S_min < ... < ladder[n-1] = S_cap < s_aggr <= s_total, and snap returns the ladder value
 * nearest to its argument (the lower one on a tie).  Hysteresis (Sec. 4.3, last paragraph; Algorithm 1
 * step 3): while the downstream stage is active the cap changes only if s* differs from the previous cap by
 * at least delta_step SMs -- except that a previous cap above S_cap (the aggressive allocation of the steps
 * without downstream work) is always replaced by s*, so that a co-running step never runs above S_cap (Eq. 1:
 * S_cap < S_aggr) and the downstream stage is never left without SMs; when the downstream stage is inactive
 * s* = s_aggr is applied at once.  The downstream stage receives s_down = max(0, s_total - s_shared).
 * The paper leaves open: the form of the moving average and its start, the tie rule of snap, whether
 * delta_step counts SMs or ladder levels (SMs here; use the ladder's spacing for "one ladder step"), and
 * whether Bhat is updated while A == 0 (it is).
 */
#ifndef HORIZONSERVE_CONTROL_H_
#define HORIZONSERVE_CONTROL_H_

#include "horizonserve.h"

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

typedef struct hs_spatial hs_spatial_t; /* opaque, owned by the library */

typedef struct {
  uint32_t abi_version;  /* HS_ABI_VERSION */
  int32_t s_total;       /* SMs of the GPU */
  int32_t s_aggr;        /* shared-stage cap while no downstream stage is active */
  int32_t n_levels;      /* entries of ladder, 1 .. 64 */
  const int32_t *ladder; /* host, strictly ascending: S_min .. S_cap; copied by hs_spatial_create */
  double b_sat;          /* pressure at which the cap reaches S_cap, > 0 */
  double gamma;          /* weight of the newest sample, 0 < gamma <= 1 */
  int32_t delta_step;    /* smallest change of the cap that is applied while co-running, >= 0 (SMs) */
} hs_spatial_config_t;

/*
 * Creates a controller.  Errors: INVALID_ARG (NULL, wrong ABI version, ladder not strictly ascending or
 * outside 1 .. s_total, S_cap >= s_aggr, s_aggr > s_total, b_sat <= 0, gamma outside (0, 1],
 * delta_step < 0, non-finite numbers).
 */
hs_status_t hs_spatial_create(const hs_spatial_config_t *cfg, hs_spatial_t **out);

/*
 * One control step: folds `pressure` (finite, >= 0) into the moving average and returns the shared stage's
 * SM budget for the next step in *s_shared and the downstream stage's in *s_down (either may be NULL).
 * Errors: INVALID_ARG (NULL controller, negative or non-finite pressure); the state is unchanged then.
 */
hs_status_t hs_spatial_update(hs_spatial_t *ctl, int32_t downstream_active, double pressure, int32_t *s_shared,
                              int32_t *s_down);

/* The moving average and the cap in force (s_aggr before the first update).  Errors: INVALID_ARG. */
hs_status_t hs_spatial_state(const hs_spatial_t *ctl, double *bhat, int32_t *s_shared);

hs_status_t hs_spatial_destroy(hs_spatial_t *ctl);

/*
 * The offline choice of the co-running cap from a sweep of fixed SM budgets (Sec. 4.1): among the budgets
 * below s_total (full allocation is what co-running must avoid, Sec. 3.2), the smallest one whose measured
 * latency is within `tolerance` (relative, >= 0; e.g. 0.05) of the best latency among them.
 *   budgets, latency: host arrays of n entries (n >= 1), budgets distinct and in 1 .. s_total, latencies > 0.
 * *s_cap receives the answer.  Errors: INVALID_ARG (NULL, n < 1, bad values, no budget below s_total).
 */
hs_status_t hs_spatial_derive_cap(const int32_t *budgets, const double *latency, int32_t n, int32_t s_total,
                                  double tolerance, int32_t *s_cap);

/*
 * ---------------------------------------------------------------------------------------------------------
 * The temporal scheduler's view: which requests the base scheduler may see in one scheduling step
 * (Sec. 4.1 "Remaining-slack ratio", Sec. 4.2 "Shared-Stage Path Rotation"; Algorithm 1 steps 1-2).
 *
 * Per request the caller passes its path (0 short: ends after the shared stage; 1 long: activates a
 * downstream stage), its stage (0 waiting for or in prefill; 1 decode continuation), its first-response
 * deadline d and a coarse estimate rhat of the time it still needs.  One call is one scheduling step k:
 *     u = (d - now) / rhat;  protected = u < u_guard      (rhat <= 0: protected iff d <= now)
 *     when a cycle starts:  N = round(N_min + f (N_max - N_min)),  f = the protected fraction of the waiting
 *                           short-path prefills (0 if there is none); halves round up
 *     phase = short during the first N steps of the cycle, long during the following M
 *     visible = decode continuations, protected requests, prefills whose path is the phase's
 *     long-path cap: of the visible unprotected long-path prefills only the (long_cap - long_admitted) with
 *                    the earliest deadlines stay visible (ties: the lower id)
 * The caller runs its base scheduler on the visible requests and "restores" the hidden ones simply by
 * passing them again at the next step.  The paper leaves open when N takes effect (here: at the start of a
 * cycle), the rounding (nearest, halves up) and the tie rule of the cap.
 */
typedef struct hs_temporal hs_temporal_t; /* opaque, owned by the library */

typedef struct {
  uint32_t abi_version; /* HS_ABI_VERSION */
  int32_t n_min, n_max; /* short-path steps per cycle, 1 <= n_min <= n_max <= 64 (the paper: 2 and 8) */
  int32_t m;            /* long-path steps per cycle, >= 1 (the paper: 2) */
  double u_guard;       /* guard band of the slack ratio, > 0 */
  int32_t long_cap;     /* most ordinary long-path prefills that may hold shared-stage slots, >= 0 */
} hs_temporal_config_t;

typedef struct {
  int64_t id;
  int32_t path;     /* 0 short, 1 long */
  int32_t stage;    /* 0 prefill (waiting or running), 1 decode continuation */
  double deadline;  /* absolute time of the first-response deadline */
  double remaining; /* estimate of the time the request still needs to its first response */
} hs_request_view_t;

hs_status_t hs_temporal_create(const hs_temporal_config_t *cfg, hs_temporal_t **out);

/*
 * One scheduling step.  reqs: host array of n requests (n >= 0; may be NULL when n == 0); long_admitted: how
 * many ordinary long-path prefills already hold shared-stage slots; visible: host array of n bytes, receives
 * 1 for visible and 0 for hidden; phase (nullable) receives 0 / 1 for a short- / long-path phase, n_short
 * (nullable) the N in force.  Errors: INVALID_ARG (NULL, n < 0, a path or stage outside {0, 1}, non-finite
 * numbers); the rotation does not advance then.
 */
hs_status_t hs_temporal_step(hs_temporal_t *ctl, double now, const hs_request_view_t *reqs, int32_t n,
                             int32_t long_admitted, uint8_t *visible, int32_t *phase, int32_t *n_short);

hs_status_t hs_temporal_destroy(hs_temporal_t *ctl);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HORIZONSERVE_CONTROL_H_ */
