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


def test_both_arms_describe_the_same_workload_and_sample():
    """The GPU arm and the reference arm print the same `config` and size the oracle's bounded sample with the same
    function: the whole 4,096-token prefix for a default run, half of it when 25 runs were asked for (so that the
    reference arm ends within a few minutes), a quarter beyond 40 runs."""
    a = bench.workload_config("32b-4k", world=1)
    assert a["workload"] == "32b-4k" and a["prefix_tokens"] == 4096 and a["suffix_tokens"] == 512 and a["layers"] == 64
    assert a == bench.workload_config("32b-4k", world=1)
    assert bench.workload_config("32b-4k", world=8)["parallelism"] == "replicas x8"
    assert bench.oracle_sample_tokens(4096, 4096, 3, 3) == 4096
    assert bench.oracle_sample_tokens(4096, 4096, 20, 5) == 2048
    assert bench.oracle_sample_tokens(4096, 4096, 50, 5) == 1024
    assert bench.oracle_sample_tokens(128, 4096, 3, 3) == 128
    assert bench.oracle_sample_tokens(4096, 1000, 3, 3) == 1000


def test_tensor_pipe_ceiling_model():
    # 148 SMs x 8,192 bf16 flop per clock per SM (one 128 x 128 x 16 MMA per 64 cycles)
    assert 2 * 128 * 128 * 16 // 64 == bench.BF16_FLOP_PER_CLK_PER_SM
    assert bench.hw_tensor_peak_tflops(1965.0) == pytest.approx(2382.6, abs=0.5)
    assert bench.hw_tensor_peak_tflops(1282.0) == pytest.approx(1554.3, abs=0.5)


def test_step_work_adds_up():
    s = synth.SHAPES["32b"]
    w = bench.step_work(s, 4096, 512)
    flops = sum(a for a, u in w.values() if u == "flop")
    assert flops == pytest.approx(bench.prefill_flops(s, 4096))            # the classes cover the whole prefill
    assert w["pack"][0] == 2 * 32 * 64 * 2 * 32768 == w["unpack"][0]       # 128 MiB read + 128 MiB written
    assert w["decode_gemv"][0] / 1e9 == pytest.approx(62.41, abs=0.01)     # every layer's weights once
    assert w["rmsnorm"][0] == 127 * 4096 * 5120 * 6


def test_documented_commands_name_existing_cases():
    """Every `python profile_case.py <case>` and `bench.py --workload <name>` quoted in profiles/ and the documents
    names a case or workload the scripts know (the commands must stay runnable as written)."""
    import glob
    import os
    import re
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    texts = [open(f).read() for f in glob.glob(os.path.join(root, "profiles", "*.md"))]
    texts += [open(os.path.join(root, f)).read() for f in ("DESIGN.md", "README.md", "BASELINE.md")]
    text = "\n".join(texts)
    source = open(os.path.join(root, "profile_case.py")).read()
    cases = set(re.findall(r"python profile_case\.py ([a-z_]+)", text))
    assert cases, "no profile command found"
    for case in cases:
        assert f'"{case}"' in source, case
    bench_src = open(os.path.join(root, "bench.py")).read()
    for name in set(re.findall(r"bench\.py --workload ([a-z0-9-]+)", text)):
        assert name in bench.WORKLOADS or f'"{name}"' in bench_src, name
