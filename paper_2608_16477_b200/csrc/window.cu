// Host-side scalar code for choosing when to start a migration (Section 4.1 cost model, Eqs. 3-9; Section 4.2 online
// selection, Algorithm 1; Section 4.4 waste bound, Eq. 10; telemetry smoothing).  No device work, no allocation.
// A candidate window is scored by what it costs the user (interruption) and what it costs the system (state prepared
// too early); the selection scans a uniform grid of windows and keeps the cheapest, preferring shorter windows on ties.
#include <cmath>

#include "../../include/kvrebuild.h"

namespace {

double clamp0(double v) { return v > 0.0 ? v : 0.0; }

void evaluate(const kv_window_inputs &in, double t_w, kv_window_eval *e) {
  e->t_w = t_w;
  // tokens the source will have produced by the time the window opens: they are the prefix the target must rebuild
  e->l_hist = in.k_curr + in.r_d * (in.t_remain - t_w);
  e->t_hist = in.t_load + e->l_hist / in.r_p;                              // time to rebuild that prefix
  const double suffix_bytes = in.r_d * t_w * in.s_kv;                      // KV the source produces during the window
  e->t_res = clamp0(suffix_bytes / in.goodput - t_w);                      // what of it the link has not carried by the handover
  // interruption: the fixed activation cost plus whichever of rebuild and transfer is still unfinished at the handover
  e->t_sit = in.t0 + std::fmax(0.0, std::fmax(e->t_hist - t_w, e->t_res));
  e->t_early = clamp0(t_w - e->t_hist);                                    // prepared state held before it is needed
  e->cost = in.alpha * e->t_sit + (1.0 - in.alpha) * e->t_early;
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
  // no window can be longer than the time left, nor than the cap on early preparation
  const double longest = clamp0(std::fmin(t_max, in->t_remain));
  const long long n = (long long)std::floor(longest / d_t + 1e-9);
  kv_window_eval cur;
  for (long long i = 0; i <= n; ++i) {
    evaluate(*in, (double)i * d_t, &cur);
    if (i == 0 || cur.cost < best->cost) *best = cur;                      // strict "<": ties keep the shorter window
  }
  // start now once the time left has shrunk to the chosen window; otherwise wait for the next control cycle
  *trigger = (in->t_remain <= best->t_w) ? 1 : 0;
  return KV_OK;
}

double kv_window_waste_bound(double t_max, double e_early, double t_avail) {
  return clamp0(t_max + e_early - t_avail);
}

double kv_ewma(double old_value, double sample, double beta) { return beta * sample + (1.0 - beta) * old_value; }

}  // extern "C"
