"""Pins of the prefetching-window oracle: the paper's equations by hand, special cases, brute-force arg-min (no GPU)."""
import math

import numpy as np
import pytest

from oracle import window_oracle as W


def _model(**kw):
    m = dict(k_curr=3000.0, r_p=15000.0, r_d=20.0, b=300e6 / 8, s_kv=262144.0, t0=0.15, alpha=0.8)
    m.update(kw)
    return m


# ---------------------------------------------------------------- oracle pins
def test_equations_by_hand():
    # Eq. (3) with the printed per-token footprint: 20 tok/s for 2 s of a 256 KiB/token cache
    assert W.s_inc(20.0, 2.0, 262144.0) == 20 * 2 * 262144
    assert W.t_hist(3000.0, 1500.0) == 2.0 and W.t_hist(3000.0, 1500.0, t_load=0.5) == 2.5          # Eq. (4)
    # Eq. (5): 10.4858 MB over 37.5 MB/s = 0.2796 s < T_w -> nothing left on the critical path
    assert W.t_res(2.0, 20.0, 262144.0, 300e6 / 8) == 0.0
    # a slow link leaves S_inc / B - T_w behind
    assert W.t_res(2.0, 20.0, 262144.0, 1e6) == pytest.approx(20 * 2 * 262144 / 1e6 - 2.0)
    assert W.t_sit(1.0, 0.2, 2.5, 0.3) == pytest.approx(0.2 + 1.5)                                   # Eq. (6): T_hist - T_w wins
    assert W.t_sit(3.0, 0.2, 2.5, 0.7) == pytest.approx(0.2 + 0.7)                                   # T_res wins
    assert W.t_sit(3.0, 0.2, 2.5, 0.0) == 0.2                                                        # both done: SIT = T_0
    assert W.t_early(3.0, 2.5) == 0.5 and W.t_early(1.0, 2.5) == 0.0                                 # Eq. (7)
    assert W.cost(0.8, 1.7, 0.5) == pytest.approx(0.8 * 1.7 + 0.2 * 0.5)                            # Eq. (8)
    assert W.l_hist_pred(3000.0, 20.0, 5.0, 2.0) == 3060.0                                           # Eq. (9)
    assert W.waste_bound(5.0, 1.0, 2.0) == 4.0 and W.waste_bound(5.0, 1.0, 9.0) == 0.0               # Eq. (10)
    assert W.ewma(10.0, 20.0, 0.25) == 12.5


def test_special_cases_of_the_model():
    m = _model()
    # both paths finish inside the window -> SIT collapses to T_0 ("reduced to T_0")
    e = W.evaluate(2.0, t_remain=2.0, **m)
    assert e["T_hist"] < 2.0 and e["T_res"] == 0.0 and e["T_SIT"] == m["t0"]
    assert e["T_early"] == pytest.approx(2.0 - e["T_hist"])
    # zero window: nothing prepared, nothing exposed: SIT = T_0 + T_hist of the full context at handover
    e0 = W.evaluate(0.0, t_remain=2.0, **m)
    assert e0["T_res"] == 0.0 and e0["T_early"] == 0.0
    assert e0["T_SIT"] == pytest.approx(m["t0"] + (m["k_curr"] + m["r_d"] * 2.0) / m["r_p"])
    # a later trigger (smaller window) means a longer prefix, an earlier one a longer suffix
    assert W.evaluate(0.5, t_remain=2.0, **m)["L_hist"] > W.evaluate(1.5, t_remain=2.0, **m)["L_hist"]


def test_selection_against_brute_force_and_extremes():
    rng = np.random.default_rng(0)
    for _ in range(200):
        m = _model(k_curr=float(rng.integers(500, 4500)), r_p=float(rng.uniform(500, 20000)),
                   r_d=float(rng.uniform(5, 60)), b=float(rng.uniform(100e6, 500e6) / 8),
                   t0=float(rng.uniform(0.05, 0.4)), alpha=float(rng.uniform(0, 1)))
        t_remain, t_max, d_t = float(rng.uniform(0, 8)), float(rng.uniform(0.5, 6)), 0.2
        tw, trigger, ev = W.select_window(t_remain=t_remain, t_max=t_max, d_t=d_t, **m)
        grid = W.candidates(min(t_max, t_remain), d_t)
        costs = [W.evaluate(c, t_remain=t_remain, **m)["J"] for c in grid]
        assert grid[-1] <= min(t_max, t_remain) + 1e-12 and len(grid) == int(math.floor(min(t_max, t_remain) / d_t + 1e-9)) + 1
        assert ev["J"] == min(costs) and tw == grid[int(np.argmin(costs))]        # arg-min, smallest window on ties
        assert trigger == (t_remain <= tw)
    # alpha = 0 only penalises early preparation: the zero window is optimal
    tw, _, _ = W.select_window(t_remain=5.0, t_max=5.0, d_t=0.2, **_model(alpha=0.0))
    assert tw == 0.0
    # alpha = 1 only penalises interruption: the chosen window reaches SIT = T_0 when the grid allows it
    tw, _, ev = W.select_window(t_remain=5.0, t_max=5.0, d_t=0.2, **_model(alpha=1.0))
    assert ev["T_SIT"] == pytest.approx(_model()["t0"])
    # deferral vs trigger: far from handover the engine waits, at the window it fires
    tw, trig_far, _ = W.select_window(t_remain=30.0, t_max=5.0, d_t=0.2, **_model())
    assert not trig_far and tw <= 5.0
    tw2, trig_now, _ = W.select_window(t_remain=tw, t_max=5.0, d_t=0.2, **_model())
    assert trig_now or tw2 < tw


