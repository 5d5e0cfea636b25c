"""CPU oracle of the prefetching-window model and the online window selection.  TEST INFRASTRUCTURE ONLY.

Plain Python floats (fp64), each function one equation of the paper in its notation:
  Eq. (1) s_KV, Eq. (3) S_inc, Eq. (4) T_hist, Eq. (5) T_res, Eq. (6) T_SIT, Eq. (7) T_early, Eq. (8) J,
  Eq. (9) predicted prefix length and the arg-min over the candidate grid, Algorithm 1 (trigger or defer),
  Eq. (10) bound on discarded preparation, and the exponentially weighted moving average of the telemetry.
Readings where the paper is silent: candidates are {0, dT, 2 dT, ...} up to and including T_limit when it is a
multiple of dT (no extra candidate at T_limit otherwise); ties of J go to the smallest window; the smoothing
factor of the moving average is a parameter (new = beta * sample + (1 - beta) * old).
Pinned by closed forms and special cases in tests/test_window_oracle.py.
"""
from __future__ import annotations

import math


def s_inc(r_d: float, t_w: float, s_kv: float) -> float:
    """Eq. (3): incremental KV volume (bytes) produced over a window: r_d * T_w * s_KV."""
    return r_d * t_w * s_kv


def t_hist(l_hist: float, r_p: float, t_load: float = 0.0) -> float:
    """Eq. (4): T_hist = T_load + L_hist / r_p."""
    return t_load + l_hist / r_p


def t_res(t_w: float, r_d: float, s_kv: float, b: float) -> float:
    """Eq. (5): T_res = max{0, S_inc(T_w) / B - T_w}; B in bytes per second."""
    return max(0.0, s_inc(r_d, t_w, s_kv) / b - t_w)


def t_sit(t_w: float, t0: float, th: float, tr: float) -> float:
    """Eq. (6): T_SIT = T_0 + max{0, T_hist - T_w, T_res}."""
    return t0 + max(0.0, th - t_w, tr)


def t_early(t_w: float, th: float) -> float:
    """Eq. (7): T_early = max{0, T_w - T_hist}."""
    return max(0.0, t_w - th)


def cost(alpha: float, sit: float, early: float) -> float:
    """Eq. (8): J = alpha * T_SIT + (1 - alpha) * T_early."""
    return alpha * sit + (1.0 - alpha) * early


def l_hist_pred(k_curr: float, r_d: float, t_remain: float, t_w: float) -> float:
    """Eq. (9), first line: predicted prefix length when preparation starts T_remain - T_w from now."""
    return k_curr + r_d * (t_remain - t_w)


def evaluate(t_w, *, k_curr, r_p, r_d, b, s_kv, t0, alpha, t_remain, t_load=0.0):
    """J, T_SIT, T_early, T_hist, T_res of one candidate window (Eqs. 4-9)."""
    lh = l_hist_pred(k_curr, r_d, t_remain, t_w)
    th = t_hist(lh, r_p, t_load)
    tr = t_res(t_w, r_d, s_kv, b)
    sit = t_sit(t_w, t0, th, tr)
    early = t_early(t_w, th)
    return {"J": cost(alpha, sit, early), "T_SIT": sit, "T_early": early, "T_hist": th, "T_res": tr, "L_hist": lh}


def candidates(t_limit: float, d_t: float):
    n = int(math.floor(t_limit / d_t + 1e-9))
    return [i * d_t for i in range(n + 1)]


def select_window(*, t_remain, t_max, d_t, **model):
    """Algorithm 1 after admission: returns (T_w*, trigger, evaluation at T_w*)."""
    t_limit = min(t_max, t_remain)
    best, best_eval = None, None
    for t_w in candidates(max(t_limit, 0.0), d_t):
        e = evaluate(t_w, t_remain=t_remain, **model)
        if best_eval is None or e["J"] < best_eval["J"]:
            best, best_eval = t_w, e
    return best, t_remain <= best, best_eval


def waste_bound(t_max: float, e_early: float, t_avail: float) -> float:
    """Eq. (10): T_waste <= max{T_max + E_early - T_avail, 0}."""
    return max(t_max + e_early - t_avail, 0.0)


def ewma(old: float, sample: float, beta: float) -> float:
    return beta * sample + (1.0 - beta) * old
