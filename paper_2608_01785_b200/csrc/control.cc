// Spatial controller: per-step choice of the shared stage's SM budget from downstream activity and a
// smoothed memory-pressure signal (Sec. 4.3, Eq. 1; Algorithm 1 step 3 of the paper), and the offline choice
// of the co-running cap from a fixed-SM sweep (Sec. 4.1).  Host-only.
#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include "../../include/horizonserve_control.h"

struct hs_spatial {
  int32_t s_total, s_aggr, delta_step;
  std::vector<int32_t> ladder;   // S_min .. S_cap, ascending
  double b_sat, gamma;
  double bhat;                   // moving average of the pressure samples
  bool primed;                   // bhat holds at least one sample
  int32_t s_shared;              // cap in force
};

namespace {

// Ladder value nearest to `target`; the lower one when two are equally near.
int32_t snap(const std::vector<int32_t>& ladder, double target) {
  int32_t best = ladder[0];
  for (size_t i = 1; i < ladder.size(); ++i)
    if (std::fabs(double(ladder[i]) - target) < std::fabs(double(best) - target)) best = ladder[i];
  return best;
}

}  // namespace

extern "C" {

hs_status_t hs_spatial_create(const hs_spatial_config_t* cfg, hs_spatial_t** out) {
  if (!cfg || !out) return HS_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->abi_version != HS_ABI_VERSION || !cfg->ladder || cfg->n_levels < 1 || cfg->n_levels > 64)
    return HS_ERR_INVALID_ARG;
  if (cfg->s_total < 1 || cfg->s_aggr > cfg->s_total || cfg->delta_step < 0) return HS_ERR_INVALID_ARG;
  if (!std::isfinite(cfg->b_sat) || !(cfg->b_sat > 0.0)) return HS_ERR_INVALID_ARG;
  if (!std::isfinite(cfg->gamma) || !(cfg->gamma > 0.0) || cfg->gamma > 1.0) return HS_ERR_INVALID_ARG;
  for (int i = 0; i < cfg->n_levels; ++i) {
    if (cfg->ladder[i] < 1 || cfg->ladder[i] > cfg->s_total) return HS_ERR_INVALID_ARG;
    if (i > 0 && cfg->ladder[i] <= cfg->ladder[i - 1]) return HS_ERR_INVALID_ARG;
  }
  if (cfg->ladder[cfg->n_levels - 1] >= cfg->s_aggr) return HS_ERR_INVALID_ARG;   // S_cap < S_aggr
  hs_spatial* c = new (std::nothrow) hs_spatial();
  if (!c) return HS_ERR_INVALID_ARG;
  c->s_total = cfg->s_total;
  c->s_aggr = cfg->s_aggr;
  c->delta_step = cfg->delta_step;
  c->ladder.assign(cfg->ladder, cfg->ladder + cfg->n_levels);
  c->b_sat = cfg->b_sat;
  c->gamma = cfg->gamma;
  c->bhat = 0.0;
  c->primed = false;
  c->s_shared = cfg->s_aggr;
  *out = c;
  return HS_OK;
}

hs_status_t hs_spatial_update(hs_spatial_t* c, int32_t downstream_active, double pressure, int32_t* s_shared,
                              int32_t* s_down) {
  if (!c || !std::isfinite(pressure) || pressure < 0.0) return HS_ERR_INVALID_ARG;
  c->bhat = c->primed ? c->gamma * pressure + (1.0 - c->gamma) * c->bhat : pressure;
  c->primed = true;
  if (!downstream_active) {
    c->s_shared = c->s_aggr;                               // Eq. 1, A = 0: applied at once
  } else {
    double rho = c->bhat / c->b_sat;
    rho = rho < 0.0 ? 0.0 : (rho > 1.0 ? 1.0 : rho);
    const int32_t s_min = c->ladder.front(), s_cap = c->ladder.back();
    const int32_t s_star = snap(c->ladder, double(s_min) + rho * double(s_cap - s_min));
    const int32_t diff = s_star > c->s_shared ? s_star - c->s_shared : c->s_shared - s_star;
    // Hysteresis holds a cap only between ladder levels: a cap above S_cap (the aggressive allocation left over
    // from the steps without downstream work) is never kept while the downstream stage runs, because Eq. 1 bounds
    // the co-running cap by S_cap < S_aggr whatever the distance to the new level.
    if (c->s_shared > s_cap || diff >= c->delta_step) c->s_shared = s_star;
  }
  if (s_shared) *s_shared = c->s_shared;
  if (s_down) *s_down = c->s_total - c->s_shared > 0 ? c->s_total - c->s_shared : 0;
  return HS_OK;
}

hs_status_t hs_spatial_state(const hs_spatial_t* c, double* bhat, int32_t* s_shared) {
  if (!c) return HS_ERR_INVALID_ARG;
  if (bhat) *bhat = c->bhat;
  if (s_shared) *s_shared = c->s_shared;
  return HS_OK;
}

hs_status_t hs_spatial_destroy(hs_spatial_t* c) {
  if (!c) return HS_ERR_INVALID_ARG;
  delete c;
  return HS_OK;
}

hs_status_t hs_spatial_derive_cap(const int32_t* budgets, const double* latency, int32_t n, int32_t s_total,
                                  double tolerance, int32_t* s_cap) {
  if (!budgets || !latency || !s_cap || n < 1 || s_total < 1) return HS_ERR_INVALID_ARG;
  if (!std::isfinite(tolerance) || tolerance < 0.0) return HS_ERR_INVALID_ARG;
  double best = 0.0;
  bool any = false;
  for (int i = 0; i < n; ++i) {
    if (budgets[i] < 1 || budgets[i] > s_total || !std::isfinite(latency[i]) || !(latency[i] > 0.0))
      return HS_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (budgets[j] == budgets[i]) return HS_ERR_INVALID_ARG;
    if (budgets[i] < s_total && (!any || latency[i] < best)) {
      best = latency[i];
      any = true;
    }
  }
  if (!any) return HS_ERR_INVALID_ARG;                     // no budget below the full allocation
  int32_t cap = 0;
  for (int i = 0; i < n; ++i)
    if (budgets[i] < s_total && latency[i] <= best * (1.0 + tolerance) && (cap == 0 || budgets[i] < cap))
      cap = budgets[i];
  *s_cap = cap;
  return HS_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ temporal view --
struct hs_temporal {
  int32_t n_min, n_max, m, long_cap;
  double u_guard;
  int32_t n;     // short-path steps of the current cycle
  int32_t pos;   // position inside the current cycle
};

extern "C" {

hs_status_t hs_temporal_create(const hs_temporal_config_t* cfg, hs_temporal_t** out) {
  if (!cfg || !out) return HS_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->abi_version != HS_ABI_VERSION || cfg->n_min < 1 || cfg->n_max < cfg->n_min || cfg->n_max > 64 ||
      cfg->m < 1 || cfg->long_cap < 0 || !std::isfinite(cfg->u_guard) || !(cfg->u_guard > 0.0))
    return HS_ERR_INVALID_ARG;
  hs_temporal* c = new (std::nothrow) hs_temporal();
  if (!c) return HS_ERR_INVALID_ARG;
  c->n_min = cfg->n_min;
  c->n_max = cfg->n_max;
  c->m = cfg->m;
  c->long_cap = cfg->long_cap;
  c->u_guard = cfg->u_guard;
  c->n = cfg->n_min;
  c->pos = 0;
  *out = c;
  return HS_OK;
}

hs_status_t hs_temporal_step(hs_temporal_t* c, double now, const hs_request_view_t* reqs, int32_t n,
                             int32_t long_admitted, uint8_t* visible, int32_t* phase_out, int32_t* n_short) {
  if (!c || n < 0 || (n > 0 && (!reqs || !visible)) || !std::isfinite(now)) return HS_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    const hs_request_view_t& r = reqs[i];
    if ((r.path != 0 && r.path != 1) || (r.stage != 0 && r.stage != 1) || !std::isfinite(r.deadline) ||
        !std::isfinite(r.remaining))
      return HS_ERR_INVALID_ARG;
  }
  std::vector<uint8_t> prot(size_t(n) > 0 ? size_t(n) : 1);
  int short_wait = 0, short_prot = 0;
  for (int i = 0; i < n; ++i) {
    const hs_request_view_t& r = reqs[i];
    const double slack = r.deadline - now;
    prot[i] = r.remaining <= 0.0 ? slack <= 0.0 : slack / r.remaining < c->u_guard;
    if (r.path == 0 && r.stage == 0) {
      ++short_wait;
      short_prot += prot[i];
    }
  }
  if (c->pos == 0) {   // a cycle starts: the short-path share follows the protected fraction
    const double f = short_wait > 0 ? double(short_prot) / double(short_wait) : 0.0;
    c->n = int32_t(std::floor(double(c->n_min) + f * double(c->n_max - c->n_min) + 0.5));
  }
  const int32_t phase = c->pos < c->n ? 0 : 1;
  c->pos = (c->pos + 1) % (c->n + c->m);
  std::vector<int> cand;
  for (int i = 0; i < n; ++i) {
    const hs_request_view_t& r = reqs[i];
    visible[i] = r.stage == 1 || prot[i] || r.path == phase;
    if (visible[i] && r.stage == 0 && r.path == 1 && !prot[i]) cand.push_back(i);
  }
  // long-path admission cap: the earliest deadlines keep their place, ties go to the lower id
  const int room = c->long_cap - long_admitted > 0 ? c->long_cap - long_admitted : 0;
  if (int(cand.size()) > room) {
    std::sort(cand.begin(), cand.end(), [&](int a, int b) {
      if (reqs[a].deadline != reqs[b].deadline) return reqs[a].deadline < reqs[b].deadline;
      return reqs[a].id < reqs[b].id;
    });
    for (size_t k = size_t(room); k < cand.size(); ++k) visible[cand[k]] = 0;
  }
  if (phase_out) *phase_out = phase;
  if (n_short) *n_short = c->n;
  return HS_OK;
}

hs_status_t hs_temporal_destroy(hs_temporal_t* c) {
  if (!c) return HS_ERR_INVALID_ARG;
  delete c;
  return HS_OK;
}

}  // extern "C"
