// Host-only entry points: Algorithm 1 (Dynamic Rollout Budget) and the temperature scheduler
// (Eq. "tp_adj" with the cosine annealing of its target entropy).  Tiny, not on the hot path.
#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "e3.h"

extern "C" const char *e3_status_string(e3_status s) {
  switch (s) {
    case E3_OK: return "E3_OK";
    case E3_ERR_INVALID_ARG: return "E3_ERR_INVALID_ARG";
    case E3_ERR_DTYPE: return "E3_ERR_DTYPE";
    case E3_ERR_ALIGNMENT: return "E3_ERR_ALIGNMENT";
    case E3_ERR_WORKSPACE: return "E3_ERR_WORKSPACE";
    case E3_ERR_INFEASIBLE: return "E3_ERR_INFEASIBLE";
    case E3_ERR_CUDA: return "E3_ERR_CUDA";
    case E3_ERR_TIMEOUT: return "E3_ERR_TIMEOUT";
  }
  return "E3_ERR_UNKNOWN";
}

extern "C" e3_status e3_allocate_budget(const double *k, int64_t B, int32_t G, int32_t G_min, int32_t G_max,
                                        int greedy_mode, int32_t *out_G) {
  if (B < 0 || G_min < 0 || (B > 0 && (!k || !out_G)) || (greedy_mode != 0 && greedy_mode != 1))
    return E3_ERR_INVALID_ARG;
  if (G_min > G || G > G_max) return E3_ERR_INFEASIBLE;
  for (int64_t i = 0; i < B; ++i)
    if (!(k[i] >= 0.0 && k[i] <= 1.0)) return E3_ERR_INVALID_ARG;
  if (B == 0) return E3_OK;

  const double k_total = std::accumulate(k, k + B, 0.0);
  if (k_total == 0.0) {
    std::fill(out_G, out_G + B, G);
    return E3_OK;
  }
  const int64_t budget = B * static_cast<int64_t>(G);
  const int64_t spare = budget - B * static_cast<int64_t>(G_min);  // N_rem after the G_min floor
  int64_t handed = 0;
  for (int64_t i = 0; i < B; ++i) {
    const int64_t share = static_cast<int64_t>(std::floor(static_cast<double>(spare) * (k[i] / k_total)));
    const int64_t g = std::min<int64_t>(G_max, static_cast<int64_t>(G_min) + share);
    out_G[i] = static_cast<int32_t>(g);
    handed += g;
  }
  int64_t left = budget - handed;

  // hardest first; equal difficulty keeps batch order
  std::vector<int64_t> by_difficulty(B);
  std::iota(by_difficulty.begin(), by_difficulty.end(), int64_t{0});
  std::stable_sort(by_difficulty.begin(), by_difficulty.end(), [k](int64_t a, int64_t b) { return k[a] > k[b]; });

  if (greedy_mode == 0) {
    for (int64_t q : by_difficulty) {
      if (left == 0) break;
      const int64_t give = std::min<int64_t>(left, G_max - out_G[q]);
      out_G[q] += static_cast<int32_t>(give);
      left -= give;
    }
  } else {
    bool progress = true;
    while (left > 0 && progress) {
      progress = false;
      for (int64_t q : by_difficulty) {
        if (left == 0) break;
        if (out_G[q] < G_max) { ++out_G[q]; --left; progress = true; }
      }
    }
  }
  return left == 0 ? E3_OK : E3_ERR_INFEASIBLE;
}

extern "C" double e3_anneal_target(const e3_sched *s) {
  if (!s) return std::nan("");
  if (s->t < s->t_anneal || s->t_max <= s->t_anneal) return s->H_init;
  const double progress =
      std::min(1.0, static_cast<double>(s->t - s->t_anneal) / static_cast<double>(s->t_max - s->t_anneal));
  const double cosine = 0.5 * (1.0 + std::cos(3.14159265358979323846 * progress));
  return s->H_init * (s->eta + (1.0 - s->eta) * cosine);
}

extern "C" e3_status e3_update_temperature(e3_sched *s, double H_t, double *tau_next) {
  if (!s || !tau_next) return E3_ERR_INVALID_ARG;
  if (!std::isfinite(H_t) || H_t <= 0.0 || s->V < 3 || !(s->tau > 0.0) || !std::isfinite(s->tau))
    return E3_ERR_INVALID_ARG;
  if (!(s->H_init > 0.0)) {  // first batch: remember the level to hold
    s->H_init = H_t;
    s->t += 1;
    *tau_next = s->tau;
    return E3_OK;
  }
  const double alpha = e3_anneal_target(s) / H_t;
  const double ln_v = std::log(static_cast<double>(s->V));
  double tau = s->tau * (1.0 + s->tau * std::log(alpha) / (ln_v + std::log(ln_v)));
  if (!(tau > 0.0)) return E3_ERR_INVALID_ARG;
  if (s->tau_max > 0.0) tau = std::min(std::max(tau, s->tau_min), s->tau_max);
  s->tau = tau;
  s->t += 1;
  *tau_next = tau;
  return E3_OK;
}

// App. A before its last simplification: tau_1 = tau_0 (1 + tau_0 ln(alpha) / Delta), Eq. "tp_relation_1".
// x = Delta / tau_0 is taken from the measured entropy through the two-level model H = (N-1) x exp(-x):
// g(x) = ln((N-1)/H) + ln x - x is concave and falls for x > 1, so Newton steps started right of the root
// come down to it monotonically and never cross it.
extern "C" double e3_entropy_gap(double H, int64_t N) {
  if (!(H > 0.0) || !std::isfinite(H) || N < 3) return std::nan("");
  const double L = std::log((static_cast<double>(N) - 1.0) / H);
  if (!(L >= 1.0)) return std::nan("");  // H above the model's maximum (N-1)/e
  double x = 2.0 * L;                      // g(2L) = ln(2L) - L < 0: right of the root
  for (int it = 0; it < 200; ++it) {
    const double g = L + std::log(x) - x;
    const double slope = 1.0 / x - 1.0;
    if (!(slope < 0.0)) break;             // x == 1: the double root at H = (N-1)/e
    const double next = std::max(1.0, x - g / slope);
    if (!(next < x)) break;
    x = next;
  }
  return x;
}

extern "C" e3_status e3_update_temperature_gap(e3_sched *s, double H_t, double *tau_next) {
  if (!s || !tau_next) return E3_ERR_INVALID_ARG;
  if (!std::isfinite(H_t) || H_t <= 0.0 || s->V < 3 || !(s->tau > 0.0) || !std::isfinite(s->tau))
    return E3_ERR_INVALID_ARG;
  const double x = e3_entropy_gap(H_t, s->V);
  if (std::isnan(x)) return E3_ERR_INVALID_ARG;
  if (!(s->H_init > 0.0)) {
    s->H_init = H_t;
    s->t += 1;
    *tau_next = s->tau;
    return E3_OK;
  }
  const double alpha = e3_anneal_target(s) / H_t;
  double tau = s->tau * (1.0 + std::log(alpha) / x);
  if (!(tau > 0.0)) return E3_ERR_INVALID_ARG;
  if (s->tau_max > 0.0) tau = std::min(std::max(tau, s->tau_min), s->tau_max);
  s->tau = tau;
  s->t += 1;
  *tau_next = tau;
  return E3_OK;
}

// ---------------------------------------------------------------------------------------------
// Sec. 4.1 difficulty model and the G_min / G_max curriculum
// ---------------------------------------------------------------------------------------------
extern "C" e3_status e3_difficulty_accumulate(int64_t D, int64_t *n_c, double *r_c, const int64_t *question_ids,
                                              const int32_t *G, const float *rewards, int64_t B) {
  if (D < 0 || B < 0 || (D > 0 && (!n_c || !r_c)) || (B > 0 && (!question_ids || !G))) return E3_ERR_INVALID_ARG;
  int64_t total = 0;
  for (int64_t b = 0; b < B; ++b) {  // look at everything before touching the state
    if (question_ids[b] < 0 || question_ids[b] >= D || G[b] < 0) return E3_ERR_INVALID_ARG;
    total += G[b];
  }
  if (total > 0 && !rewards) return E3_ERR_INVALID_ARG;
  const float *r = rewards;
  for (int64_t b = 0; b < B; ++b) {
    double sum = 0.0;
    for (int32_t j = 0; j < G[b]; ++j) sum += static_cast<double>(r[j]);
    r += G[b];
    r_c[question_ids[b]] += sum;
    n_c[question_ids[b]] += G[b];
  }
  return E3_OK;
}

extern "C" e3_status e3_difficulty_rank(int64_t D, const int64_t *n_c, const double *r_c, double *out_k) {
  if (D < 0 || (D > 0 && (!n_c || !r_c || !out_k))) return E3_ERR_INVALID_ARG;
  std::vector<double> avg(static_cast<size_t>(D));
  for (int64_t i = 0; i < D; ++i) {
    if (n_c[i] < 0 || !std::isfinite(r_c[i])) return E3_ERR_INVALID_ARG;
    avg[i] = n_c[i] > 0 ? r_c[i] / static_cast<double>(n_c[i]) : 0.0;
  }
  std::vector<int64_t> order(static_cast<size_t>(D));
  std::iota(order.begin(), order.end(), int64_t(0));
  std::stable_sort(order.begin(), order.end(), [&](int64_t a, int64_t b) { return avg[a] > avg[b]; });
  for (int64_t pos = 0; pos < D; ++pos) out_k[order[pos]] = static_cast<double>(pos + 1) / static_cast<double>(D);
  return E3_OK;
}

extern "C" e3_status e3_budget_curriculum(int32_t G, int32_t step, int32_t G_min_limit, int32_t G_max_limit,
                                          int64_t epochs_done, int32_t *G_min, int32_t *G_max) {
  if (!G_min || !G_max || G < 0 || step < 0 || epochs_done < 0 || G_min_limit < 0) return E3_ERR_INVALID_ARG;
  if (G_min_limit > G || G_max_limit < G) return E3_ERR_INFEASIBLE;
  // closed form of "widen by `step` per finished epoch until the limit"
  const int64_t moved = static_cast<int64_t>(step) * epochs_done;  // step, epochs_done >= 0
  const int64_t up = static_cast<int64_t>(G_max_limit) - G, down = static_cast<int64_t>(G) - G_min_limit;
  *G_max = static_cast<int32_t>(G + (step > 0 && epochs_done > up / step ? up : std::min(moved, up)));
  *G_min = static_cast<int32_t>(G - (step > 0 && epochs_done > down / step ? down : std::min(moved, down)));
  return E3_OK;
}

