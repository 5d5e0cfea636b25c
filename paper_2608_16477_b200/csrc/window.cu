// Host-side scalar code of the Scheduler Engine: the prefetching-window cost model (Eqs. 3-9), the grid search
// and trigger decision of Algorithm 1, the waste bound of Eq. (10) and the telemetry smoothing.  No device work.
#include <cmath>

#include "../../include/kvrebuild.h"

namespace {

double clamp0(double v) { return v > 0.0 ? v : 0.0; }

void evaluate(const kv_window_inputs &in, double t_w, kv_window_eval *e) {
  e->t_w = t_w;
  e->l_hist = in.k_curr + in.r_d * (in.t_remain - t_w);                    // Eq. (9), predicted prefix length
  e->t_hist = in.t_load + e->l_hist / in.r_p;                              // Eq. (4)
  const double s_inc = in.r_d * t_w * in.s_kv;                             // Eq. (3)
  e->t_res = clamp0(s_inc / in.goodput - t_w);                             // Eq. (5)
  e->t_sit = in.t0 + std::fmax(0.0, std::fmax(e->t_hist - t_w, e->t_res)); // Eq. (6)
  e->t_early = clamp0(t_w - e->t_hist);                                    // Eq. (7)
  e->cost = in.alpha * e->t_sit + (1.0 - in.alpha) * e->t_early;           // Eq. (8)
}

bool valid(const kv_window_inputs *in) {
  return in != nullptr && in->r_p > 0.0 && in->r_d >= 0.0 && in->goodput > 0.0 && in->s_kv > 0.0 && in->k_curr >= 0.0 &&
         in->alpha >= 0.0 && in->alpha <= 1.0 && in->t0 >= 0.0 && in->t_load >= 0.0 && std::isfinite(in->t_remain);
}

}  // namespace

extern "C" {

int32_t kv_window_evaluate(const kv_window_inputs *in, double t_w, kv_window_eval *out) {
  if (!valid(in) || out == nullptr || !(t_w >= 0.0)) return KV_ERR_ARG;
  evaluate(*in, t_w, out);
  return KV_OK;
}

int32_t kv_window_select(const kv_window_inputs *in, double t_max, double d_t, kv_window_eval *best, int32_t *trigger) {
  if (!valid(in) || best == nullptr || trigger == nullptr || !(d_t > 0.0) || !(t_max >= 0.0)) return KV_ERR_ARG;
  const double t_limit = clamp0(std::fmin(t_max, in->t_remain));           // T_limit = min(T_max, T_remain)
  const long long n = (long long)std::floor(t_limit / d_t + 1e-9);
  kv_window_eval cur;
  for (long long i = 0; i <= n; ++i) {                                     // W = {0, dT, ..., T_limit}
    evaluate(*in, (double)i * d_t, &cur);
    if (i == 0 || cur.cost < best->cost) *best = cur;                      // ties keep the smaller window
  }
  *trigger = (in->t_remain <= best->t_w) ? 1 : 0;                          // trigger iff T_remain <= T_w*
  return KV_OK;
}

double kv_window_waste_bound(double t_max, double e_early, double t_avail) {
  return clamp0(t_max + e_early - t_avail);                                // Eq. (10)
}

double kv_ewma(double old_value, double sample, double beta) { return beta * sample + (1.0 - beta) * old_value; }

}  // extern "C"
