"""Host-side arithmetic of bench.py: the executed-flop count behind the TFLOP/s figures and the roofline peaks."""
import pytest

import bench
import synth


def test_prefill_flops_match_the_algorithmic_work():
    s = synth.SHAPES["32b"]
    # per-token linear work L * [2 D (Hq + 2 Hkv) d + 2 Hq d D + 6 D F], causal attention 2 Hq d N (N + 1) L
    n = 4096
    linear = s.n_layers * (2 * s.hidden * (s.q_dim + 2 * s.kv_dim) + 2 * s.q_dim * s.hidden + 6 * s.hidden * s.ffn) * n
    attn = 2 * s.n_q_heads * s.head_dim * n * (n + 1) * s.n_layers
    assert linear / 1e12 == pytest.approx(255.637, abs=1e-3)
    assert attn / 1e12 == pytest.approx(17.597, abs=1e-3)
    assert bench.prefill_flops(s, n, with_logits=True) == pytest.approx(linear + attn)
    # K/V-only prefill: the last layer stops after its QKV projection
    assert bench.prefill_flops(s, n) / 1e12 == pytest.approx(269.39, abs=5e-3)


def test_sweep_and_8b_totals():
    s = synth.SHAPES["32b"]
    for n, total in ((512, 32.230), (2048, 132.218), (8192, 581.650), (16384, 1304.038)):
        assert bench.prefill_flops(s, n, with_logits=True) / 1e12 == pytest.approx(total, abs=2e-3)
    assert bench.prefill_flops(synth.SHAPES["8b"], 1024, with_logits=True) / 1e12 == pytest.approx(14.535, abs=2e-3)


def test_peaks_have_every_key():
    p = bench.peaks()
    assert p["source"] in ("measured", "fallback")
    assert p["hbm_gbs"] > 0 and p["bf16_tflops"] >= p["bf16_tflops_sustained"] > 0
