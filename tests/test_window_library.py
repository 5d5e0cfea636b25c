"""The library's host-side window model and selection against the oracle on seeded random inputs (no GPU)."""
import numpy as np
import pytest

from oracle import window_oracle as W
from tests.test_window_oracle import _model


# ---------------------------------------------------------------- library host code == oracle
def test_library_matches_oracle():
    import paper_2608_16477_b200 as kv
    kv.load()
    rng = np.random.default_rng(1)
    for _ in range(300):
        m = _model(k_curr=float(rng.integers(100, 9000)), r_p=float(rng.uniform(300, 30000)),
                   r_d=float(rng.uniform(0, 80)), b=float(rng.uniform(50e6, 1e9) / 8),
                   t0=float(rng.uniform(0, 0.5)), alpha=float(rng.uniform(0, 1)))
        t_remain, t_max, d_t = float(rng.uniform(0, 10)), float(rng.uniform(0.1, 6)), float(rng.choice([0.1, 0.2, 0.5]))
        lib_in = dict(k_curr=m["k_curr"], r_p=m["r_p"], r_d=m["r_d"], goodput=m["b"], s_kv=m["s_kv"], t0=m["t0"],
                      t_load=0.0, alpha=m["alpha"], t_remain=t_remain)
        tw, trigger, ev = W.select_window(t_remain=t_remain, t_max=t_max, d_t=d_t, **m)
        got, got_trigger = kv.kv_window_select(t_max, d_t, **lib_in)
        assert got["t_w"] == pytest.approx(tw, abs=1e-12) and got_trigger == trigger
        for a, b in (("cost", "J"), ("t_sit", "T_SIT"), ("t_early", "T_early"), ("t_hist", "T_hist"),
                     ("t_res", "T_res"), ("l_hist", "L_hist")):
            assert got[a] == pytest.approx(ev[b], rel=1e-12, abs=1e-12)
        one = kv.kv_window_evaluate(0.7, **lib_in)
        ref = W.evaluate(0.7, t_remain=t_remain, **m)
        assert one["cost"] == pytest.approx(ref["J"], rel=1e-12, abs=1e-12)
    assert kv.kv_window_waste_bound(5.0, 1.0, 2.0) == 4.0 and kv.kv_ewma(10.0, 20.0, 0.25) == 12.5
    from paper_2608_16477_b200 import KVError
    with pytest.raises(KVError):
        kv.kv_window_select(5.0, 0.0, **lib_in)            # dT must be positive
