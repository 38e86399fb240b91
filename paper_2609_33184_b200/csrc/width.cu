// I/O-aware dynamic verification width (Section 4.2): q* = argmin over the candidate widths of
// T_round(q) / U(q), estimated from the recent rounds at each width.  Host logic only.
//
// Readings where the paper gives no formula: per-width running means are exponential moving
// averages; the verification cost counts overlapped transfer and compute once,
// T_V = max(t_transfer, t_compute); an initial sampling phase visits every width
// `sample_rounds` times (in the order of the candidate list) before any estimate is trusted;
// afterwards the width changes only if the best width's estimated cost per committed token is
// lower than the current width's by more than `switch_threshold` (relative).  Ties keep the
// smaller width.
#include <new>

#include "specstream.h"

struct ss_width {
  ss_width_config cfg;
  double t_draft[8], t_verify[8], t_other[8], u[8];
  int32_t n_obs[8];
  int32_t current;  // index into cfg.widths
};

namespace {
int find_width(const ss_width* w, int32_t q) {
  for (int i = 0; i < w->cfg.n_widths; ++i)
    if (w->cfg.widths[i] == q) return i;
  return -1;
}
double cost_of(const ss_width* w, int i) {
  const double t = w->t_draft[i] + w->t_verify[i] + w->t_other[i];
  return w->u[i] > 0.0 ? t / w->u[i] : 1e300;
}
}  // namespace

extern "C" {

ss_status ss_width_create(ss_width** out, const ss_width_config* cfg) {
  if (!out || !cfg) return SS_ERR_ARG;
  if (cfg->n_widths <= 0 || cfg->n_widths > 8 || cfg->sample_rounds < 1 || !(cfg->ema > 0.f) ||
      cfg->ema > 1.f || cfg->switch_threshold < 0.f)
    return SS_ERR_ARG;
  for (int i = 0; i < cfg->n_widths; ++i) {
    if (cfg->widths[i] <= 0) return SS_ERR_ARG;
    for (int j = 0; j < i; ++j)
      if (cfg->widths[j] == cfg->widths[i]) return SS_ERR_ARG;
  }
  ss_width* w = new (std::nothrow) ss_width();
  if (!w) return SS_ERR_ARG;
  *w = ss_width{};
  w->cfg = *cfg;
  *out = w;
  return SS_OK;
}

ss_status ss_width_destroy(ss_width* w) {
  if (!w) return SS_ERR_ARG;
  delete w;
  return SS_OK;
}

ss_status ss_width_observe(ss_width* w, int32_t q, const ss_width_obs* o) {
  if (!w || !o) return SS_ERR_ARG;
  const int i = find_width(w, q);
  if (i < 0 || o->committed < 0 || o->t_draft < 0.f || o->t_transfer < 0.f || o->t_compute < 0.f ||
      o->t_other < 0.f)
    return SS_ERR_ARG;
  // overlapped transfer and compute are counted once
  const double tv = (double)(o->t_transfer > o->t_compute ? o->t_transfer : o->t_compute);
  const double a = w->n_obs[i] == 0 ? 1.0 : (double)w->cfg.ema;
  w->t_draft[i] += a * ((double)o->t_draft - w->t_draft[i]);
  w->t_verify[i] += a * (tv - w->t_verify[i]);
  w->t_other[i] += a * ((double)o->t_other - w->t_other[i]);
  w->u[i] += a * ((double)o->committed - w->u[i]);
  ++w->n_obs[i];
  return SS_OK;
}

int32_t ss_width_next(ss_width* w) {
  if (!w) return -1;
  // sampling phase: the first width (in list order) that has not been tried often enough
  for (int i = 0; i < w->cfg.n_widths; ++i)
    if (w->n_obs[i] < w->cfg.sample_rounds) {
      w->current = i;
      return w->cfg.widths[i];
    }
  int best = 0;
  for (int i = 1; i < w->cfg.n_widths; ++i) {
    const double ci = cost_of(w, i), cb = cost_of(w, best);
    if (ci < cb || (ci == cb && w->cfg.widths[i] < w->cfg.widths[best])) best = i;
  }
  const double cur = cost_of(w, w->current), bst = cost_of(w, best);
  if (best != w->current && bst < cur * (1.0 - (double)w->cfg.switch_threshold)) w->current = best;
  return w->cfg.widths[w->current];
}

ss_status ss_width_estimate(ss_width* w, int32_t q, double* t_round, double* committed, double* cost,
                            int32_t* n_obs) {
  if (!w) return SS_ERR_ARG;
  const int i = find_width(w, q);
  if (i < 0) return SS_ERR_ARG;
  if (t_round) *t_round = w->t_draft[i] + w->t_verify[i] + w->t_other[i];
  if (committed) *committed = w->u[i];
  if (cost) *cost = cost_of(w, i);
  if (n_obs) *n_obs = w->n_obs[i];
  return SS_OK;
}

}  // extern "C"
