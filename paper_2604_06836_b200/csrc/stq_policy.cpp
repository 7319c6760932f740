// Host-side transition decision (Sec. 3.3-3.4; Algorithm 1, decision branch).  O(L) per decision,
// three scalars of state: this is the "linear-time" replacement for a search over widths.
#include <cmath>
#include <new>
#include <vector>

#include "../../include/stq.h"

struct stq_policy {
  stq_policy_cfg cfg;
  double n_bar = 0.0, r_bar = 0.0, v_bar = 0.0;   // global running statistics (start at 0)
};

namespace {
const double kPhi = 7.2;                       // base bias: an average layer lands on 8 bits
const double kCut4 = 6.8, kCut8 = 12.0, kCut16 = 24.0;
const int64_t kEarlySteps = 5;                 // decide on every step t < 5

uint8_t map_score(double s) {
  if (s < kCut4) return 4;
  if (s < kCut8) return 8;
  if (s < kCut16) return 16;
  return 32;
}
}  // namespace

extern "C" {

int stq_policy_create(stq_policy** out, const stq_policy_cfg* cfg) {
  if (!out || !cfg) return STQ_E_NULL;
  *out = nullptr;
  if (!(cfg->alpha >= 0.0 && cfg->alpha <= 1.0) || !(cfg->tau > 0.0) || !(cfg->eps_stat >= 0.0) ||
      cfg->interval < 1)
    return STQ_E_ARG;
  stq_policy* p = new (std::nothrow) stq_policy();
  if (!p) return STQ_E_WORKSPACE;
  p->cfg = *cfg;
  *out = p;
  return STQ_OK;
}

int stq_policy_destroy(stq_policy* p) {
  if (!p) return STQ_E_NULL;
  delete p;
  return STQ_OK;
}

int stq_policy_is_decision_step(const stq_policy* p, int64_t t) {
  if (!p) return 0;
  return (t % p->cfg.interval == 0 || t < kEarlySteps) ? 1 : 0;
}

int stq_decide(stq_policy* p, const double* stats, int L, int64_t t, uint8_t* bits_out, double* score_out) {
  if (!p || !stats || !bits_out) return STQ_E_NULL;
  if (L <= 0) return STQ_E_NUMEL;
  const double eps = p->cfg.eps_stat;
  std::vector<double> n(L), r(L), v(L);
  double acc_n = 0.0, acc_r = 0.0, acc_v = 0.0;
  for (int l = 0; l < L; ++l) {
    const double sum_g = stats[4 * l], sum_abs = stats[4 * l + 1], sum_sq = stats[4 * l + 2];
    const double count = stats[4 * l + 3];
    if (!(count > 0.0)) return STQ_E_ARG;
    const double ms = sum_sq / count;            // hierarchical factor v_l (Eq. 8)
    const double mu_abs = sum_abs / count;
    const double centre = p->cfg.cv_of_signed ? sum_g / count : mu_abs;
    double var = ms - centre * centre;
    if (var < 0.0) var = 0.0;
    v[l] = ms;
    n[l] = std::sqrt(ms);                        // intensity factor (Eq. 2)
    r[l] = std::sqrt(var) / (mu_abs + eps);      // variation factor (Eq. 3)
    acc_n += n[l]; acc_r += r[l]; acc_v += v[l];
  }
  const double a = p->cfg.alpha;
  p->n_bar = a * (acc_n / L) + (1.0 - a) * p->n_bar;
  p->r_bar = a * (acc_r / L) + (1.0 - a) * p->r_bar;
  p->v_bar = a * (acc_v / L) + (1.0 - a) * p->v_bar;
  const double anneal = 1.0 + 1.0 / std::cosh((double)t / p->cfg.tau);   // Eq. 7
  const double log_anneal = std::log2(anneal);
  for (int l = 0; l < L; ++l) {
    const double score = kPhi + std::log2(r[l] / (p->r_bar + eps)) + std::log2(n[l] / (p->n_bar + eps)) +
                         log_anneal + std::log2(v[l] / (p->v_bar + eps));
    if (score_out) score_out[l] = score;
    bits_out[l] = map_score(score);
  }
  return STQ_OK;
}

int stq_policy_get_state(const stq_policy* p, double out[3]) {
  if (!p || !out) return STQ_E_NULL;
  out[0] = p->n_bar; out[1] = p->r_bar; out[2] = p->v_bar;
  return STQ_OK;
}

int stq_policy_set_state(stq_policy* p, const double in[3]) {
  if (!p || !in) return STQ_E_NULL;
  p->n_bar = in[0]; p->r_bar = in[1]; p->v_bar = in[2];
  return STQ_OK;
}

}  // extern "C"
