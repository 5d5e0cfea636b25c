#!/usr/bin/env python
"""Benchmark of the KV-rebuild hot path on B200: prefix prefill into a paged cache, suffix pack,
unpack/assemble and the resumed decode step, through the C ABI.

  python bench.py --gpus N --steps K --warmup W            (N > 1: launched by torch.distributed.run)
  python bench.py --impl reference ...                     (the CPU oracle on a bounded sample)
  python bench.py --workload pack-stress | stream-overlap | batched-prefill
                                                           (side measurements: copy steady state, suffix streaming
                                                            under decode, concurrent migrations; one GPU)

One "step" is one pass of the whole path for one request of the workload.  Every rank runs an independent
replica (the path does not shard: no data-path collective), so scaling is weak and `value` is the sum of
the ranks' prefix tokens divided by the slowest rank's time.  Prints ONE JSON line on rank 0.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "prefix_kv_rebuild_tokens_per_s"
UNIT = "tokens/s"
# profiling recipe fallbacks when MEASURED_PEAKS.json is absent
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0

WORKLOADS = {
    # name: (shape, prefix tokens, suffix tokens, pool blocks)
    "32b-4k": ("32b", 4096, 512, 4096),
    # prefix-length sweep of the same shape, suffix = prefix / 8 (parity cases / context; not the bench line)
    "32b-512": ("32b", 512, 64, 4096),
    "32b-2k": ("32b", 2048, 256, 4096),
    "32b-8k": ("32b", 8192, 1024, 4096),
    "32b-16k": ("32b", 16384, 2048, 4096),
    "8b-1k": ("8b", 1024, 256, 1024),
    "tiny": ("tiny", 128, 32, 64),
}

# DRAM bytes (read + write) of one gate/up GEMM launch at the 32b-4k workload, from the ncu capture
# summarised under profiles/ (same shape as the bench's launch: M 4096, K 5120, 2 x 25600 weight rows).
NCU_TRAFFIC_BYTES = {"32b-4k": 1269.9e6}   # profiles/gemm_tc_pair_gate_up_32b-4k.md: 1,064.3 MB read + 205.6 MB written


# Tensor-pipe arithmetic of one B200 SM: a 128 x 128 x 16 bf16 tcgen05.mma retires in 64 cycles
# (2 * 128 * 128 * 16 / 64 = 8,192 flop per clock per SM; a probe of back-to-back MMAs measured 67 cycles).
SM_COUNT = 148
BF16_FLOP_PER_CLK_PER_SM = 8192
NOMINAL_BF16_TFLOPS = 2250.0      # datasheet dense bf16 figure


def hw_tensor_peak_tflops(sm_mhz):
    """Tensor-pipe ceiling at a given SM clock: SMs x flop/clk/SM x clock."""
    return SM_COUNT * BF16_FLOP_PER_CLK_PER_SM * sm_mhz * 1e6 / 1e12


def workload_config(workload, world=1, layers=0):
    """The `config` object of the JSON line, the same in both arms."""
    shape_name, prefix, suffix, pool_blocks = WORKLOADS[workload]
    shape = synth.SHAPES[shape_name]
    return {"workload": workload, "shape": shape.name, "layers": layers or shape.n_layers,
            "prefix_tokens": prefix, "suffix_tokens": suffix, "block_size": shape.block_size, "pool_blocks": pool_blocks,
            "block_ids": "seeded permutation (fragmented)", "parallelism": f"replicas x{world}",
            "l2": "inputs larger than L2: each step streams every weight (>> 126 MB) between "
                  "consecutive launches of any kernel; standalone pack/unpack rotate over disjoint block sets"}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": FALLBACK_BF16_TFLOPS_SUSTAINED, "source": "fallback"}


def prefill_flops(shape, n_tokens, with_logits=False):
    """Executed flops of a K/V-only prefill: the last layer stops after its QKV projection."""
    d, qd, kvd, f, L = shape.hidden, shape.q_dim, shape.kv_dim, shape.ffn, shape.n_layers
    qkv = 2.0 * n_tokens * d * (qd + 2 * kvd)
    rest = 2.0 * n_tokens * (qd * d + 3 * d * f)
    attn = 2.0 * shape.n_q_heads * shape.head_dim * n_tokens * (n_tokens + 1)   # causal: N(N+1)/2 pairs, QK and PV
    full_layers = L if with_logits else L - 1
    return L * qkv + full_layers * (rest + attn)


def step_work(shape, prefix, suffix):
    """Algorithmic work of one bench step per kernel class: (amount, unit) with flops for the tensor-bound classes
    and bytes (read + written) for the HBM-bound ones.  K/V-only prefill: the last layer stops after its QKV projection."""
    d, qd, kvd, f, L = shape.hidden, shape.q_dim, shape.kv_dim, shape.ffn, shape.n_layers
    n = prefix
    n_ctx = prefix + suffix + 1
    page_payload = -(-suffix // shape.block_size) * L * 2 * synth.kv_page_bytes(shape)
    return {
        "gemm_qkv": (L * 2.0 * n * d * (qd + 2 * kvd), "flop"),
        "attention": ((L - 1) * 2.0 * shape.n_q_heads * shape.head_dim * n * (n + 1), "flop"),
        "gemm_o": ((L - 1) * 2.0 * n * qd * d, "flop"),
        "gemm_gate_up": ((L - 1) * 2.0 * n * d * 2 * f, "flop"),
        "gemm_down": ((L - 1) * 2.0 * n * f * d, "flop"),
        "rmsnorm": ((2 * L - 1) * n * d * 6.0, "byte"),
        "pack": (2.0 * page_payload, "byte"),
        "unpack": (2.0 * page_payload, "byte"),
        "decode_gemv": (L * 2.0 * (d * (qd + 2 * kvd) + qd * d + 3 * d * f), "byte"),
        "decode_attention": (L * 2.0 * n_ctx * kvd * 2, "byte"),
        "lm_head": (2.0 * shape.vocab * d, "byte"),
    }


# ------------------------------------------------------------------------------------------ reference arm
def oracle_sample(shape, n_tokens, prefix=None, seed=0):
    """Bounded sample of the workload for the CPU oracle: ONE decoder layer over n_tokens rows of the prefix.  When the
    sample is shorter than the prefix it is the MIDDLE of it (rows (prefix - n) / 2 ... attending to the cached rows
    before them), so that a row sees as many keys on average as a row of the whole prefix does and attention keeps
    its true share of the work."""
    from oracle import kv_oracle as O
    prefix = n_tokens if prefix is None else prefix
    start = (prefix - n_tokens) // 2
    w = synth.layer_weights(shape, seed, 0)
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n_tokens, shape.hidden)) * shape.init_std
    k_past = rng.standard_normal((start, shape.n_kv_heads, shape.head_dim)) if start else None
    v_past = rng.standard_normal((start, shape.n_kv_heads, shape.head_dim)) if start else None
    pos = np.arange(start, start + n_tokens)

    def run():
        t0 = time.perf_counter()
        O.layer_forward(shape, w, x, pos, k_past=k_past, v_past=v_past)
        return time.perf_counter() - t0
    return run


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_copy_rates(shape, n_blocks):
    """The oracle's pack and unpack/assemble over n_blocks scattered pages, in GB/s (bytes read + bytes written)."""
    from oracle import kv_oracle as O
    pool = 2 * n_blocks + 8
    cache = O.new_cache(shape.n_layers, pool, shape.block_size, shape.n_kv_heads, shape.head_dim, fill=1)
    ids = np.random.default_rng(5).permutation(pool)
    src, dst = ids[:n_blocks], ids[n_blocks:2 * n_blocks]
    t0 = time.perf_counter()
    wire = O.pack_blocks(cache, src)
    t1 = time.perf_counter()
    st, _ = O.unpack_assemble(cache, wire, np.arange(n_blocks), dst, [], n_blocks * shape.block_size)
    t2 = time.perf_counter()
    assert st == O.OK
    return 2.0 * wire.nbytes / (t1 - t0) / 1e9, 2.0 * wire.nbytes / (t2 - t1) / 1e9


def oracle_sample_tokens(prefix, cap, steps, warmup):
    """Prefix tokens in the oracle's bounded sample: the whole prefix when the steps + warm-ups asked for fit in about
    four minutes of host time (one layer over 4,096 tokens of the 32B shape takes about 17 s on 16 cores), else half
    or a quarter of it.  Both arms size the sample with this function, so they time the same work."""
    tokens = min(prefix, cap)
    runs = steps + warmup
    if runs > 13:
        tokens = min(tokens, max(prefix // 2, 1))
    if runs > 40:
        tokens = min(tokens, max(prefix // 4, 1))
    return tokens


def oracle_sample_text(shape, prefix, sample_tokens):
    part = ("the whole prefix" if sample_tokens == prefix else
            f"the middle {sample_tokens} of {prefix} prefix tokens (rows {(prefix - sample_tokens) // 2} to "
            f"{(prefix + sample_tokens) // 2 - 1}, attending to the cached rows before them: the same mean number of "
            f"keys per row as over the whole prefix)")
    return (f"one decoder layer (1 of {shape.n_layers}) of the fp64 numpy oracle over {part}; tokens/s extrapolated "
            f"to {shape.n_layers} layers")


def cpu_baseline(shape, prefix, sample_tokens, repeats=3, suffix_blocks=0):
    """The oracle as it stands on the host cores: best of `repeats` runs of the bounded sample."""
    run = oracle_sample(shape, sample_tokens, prefix)
    times = [run() for _ in range(repeats)]
    secs = min(times)
    value = sample_tokens / (secs * shape.n_layers)
    extra = {}
    if suffix_blocks:
        pack, unpack = oracle_copy_rates(shape, suffix_blocks)
        extra = {"pack_gbs": pack, "unpack_gbs": unpack, "copy_sample": f"{suffix_blocks} suffix blocks, one thread"}
    return {**extra, "value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": oracle_sample_text(shape, prefix, sample_tokens) + f"; best of {repeats} runs",
            "seconds": secs, "seconds_all": [round(t, 3) for t in times]}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    shape_name, prefix, suffix, _ = WORKLOADS[args.workload]
    shape = synth.SHAPES[shape_name]
    warmup = max(args.ref_warmup, args.warmup if args.warmup_given else 0)
    sample_tokens = oracle_sample_tokens(prefix, args.ref_tokens, args.steps, warmup)
    run = oracle_sample(shape, sample_tokens, prefix)
    for _ in range(warmup):
        run()
    times = [run() for _ in range(args.steps)]
    secs = sum(times) / len(times)
    value = sample_tokens / (secs * shape.n_layers)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": warmup, "ms_per_step": secs * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args.workload, world=args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": oracle_sample_text(shape, prefix, sample_tokens) + f"; mean of {args.steps} steps",
                         "best_value": sample_tokens / (min(times) * shape.n_layers)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1])); mx.append(float(p[2])); power.append(float(p[3]))
                except ValueError:
                    continue
                for name, val in zip(names, p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": float(max(power))}


# ------------------------------------------------------------------------------------------ our arm
def build_model(kv, torch, shape, seed=1000):
    """Random-init weights of the shape, N(0, init_std^2) in bf16, norm gains 1, created on the device."""
    gen = torch.Generator(device="cuda").manual_seed(seed)

    def mat(rows, cols):
        return torch.empty(rows, cols, dtype=torch.bfloat16, device="cuda").normal_(0.0, shape.init_std, generator=gen)

    def layer(l):
        ones = torch.ones(shape.hidden, dtype=torch.bfloat16, device="cuda")
        return {"attn_norm": ones, "ffn_norm": ones.clone(), "w_qkv": mat(shape.qkv_dim, shape.hidden),
                "w_o": mat(shape.hidden, shape.q_dim), "w_gate_up": mat(2 * shape.ffn, shape.hidden),
                "w_down": mat(shape.hidden, shape.ffn)}
    head = {"embed": mat(shape.vocab, shape.hidden), "lm_head": mat(shape.vocab, shape.hidden),
            "final_norm": torch.ones(shape.hidden, dtype=torch.bfloat16, device="cuda")}
    return kv.Model(shape, head, layer), gen


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2608_16477_b200 as kv
    from paper_2608_16477_b200 import replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    kv.load()

    shape_name, prefix, suffix, pool_blocks = WORKLOADS[args.workload]
    shape = synth.SHAPES[shape_name]
    if args.layers:
        shape = shape.with_layers(args.layers)
    bs = shape.block_size
    n = prefix + suffix
    seed = 1000 + rank
    model, gen = build_model(kv, torch, shape, seed)

    ids = synth.token_ids(shape, seed, n + 1)
    src = kv.PagedCache(shape, pool_blocks)
    tgt = kv.PagedCache(shape, pool_blocks, fill=0)
    kv.kv_fill_pattern(src.data, src.data.numel() * 2, seed=seed)        # source pool holds arbitrary KV bytes
    perm_src = synth.block_permutation(seed + 1, pool_blocks)
    perm_tgt = synth.block_permutation(seed + 2, pool_blocks)
    nb_prefix, nb_total = prefix // bs, -(-n // bs)
    nb_suffix = nb_total - nb_prefix
    tgt_prefix = perm_tgt[:nb_prefix].copy()
    dst_ids = perm_tgt[nb_prefix:nb_total].copy()
    extra = [int(perm_tgt[nb_total])] if n % bs == 0 else []
    logical = np.arange(nb_prefix, nb_total, dtype=np.int32)
    src_suffix = perm_src[nb_prefix:nb_total].copy()
    wire_elems = nb_suffix * shape.n_layers * 2 * (src.page_bytes // 2)
    wire = torch.empty(wire_elems, dtype=torch.int16, device="cuda")
    wire2 = torch.empty_like(wire)
    wire_host = torch.empty(wire_elems, dtype=torch.int16, pin_memory=True)
    logits = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    logits_host = torch.empty(shape.vocab, dtype=torch.float32, pin_memory=True)
    ws_p = model.workspace(kv.KV_OP_PREFILL, prefix)
    ws_d = model.workspace(kv.KV_OP_DECODE, n + 1)
    stream = torch.cuda.current_stream()

    def step():
        kv.kv_prefill_prefix(model, tgt, ids[:prefix], tgt_prefix, workspace=ws_p)
        kv.kv_pack_blocks(src, src_suffix, wire)
        merged = kv.kv_unpack_assemble(tgt, wire, logical, dst_ids, tgt_prefix, n, epoch=1, expected_epoch=1)
        kv.kv_decode_step(model, tgt, int(ids[n]), n, list(merged) + extra, logits, workspace=ws_d)

    e2e_marks = []
    side = torch.cuda.Stream()

    def step_e2e():
        # host buffers: token ids and tables are host arrays; the wire crosses the host (the link between source and
        # target) and the logits are read back.  As in the method itself, the suffix travels WHILE the target rebuilds
        # the prefix (parallel preparation): pack, device-to-host and host-to-device copies run on a side stream beside
        # the prefill; assembly waits for both.  Events split the step into its legs.
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        ev[0].record(stream)
        side.wait_stream(stream)
        ev[4].record(side)
        kv.kv_pack_blocks(src, src_suffix, wire, stream=side)
        with torch.cuda.stream(side):
            wire_host.copy_(wire, non_blocking=True)
            wire2.copy_(wire_host, non_blocking=True)
        ev[5].record(side)
        kv.kv_prefill_prefix(model, tgt, ids[:prefix], tgt_prefix, workspace=ws_p)
        ev[1].record(stream)
        stream.wait_stream(side)
        merged = kv.kv_unpack_assemble(tgt, wire2, logical, dst_ids, tgt_prefix, n, epoch=1, expected_epoch=1)
        kv.kv_decode_step(model, tgt, int(ids[n]), n, list(merged) + extra, logits, workspace=ws_d)
        ev[2].record(stream)
        logits_host.copy_(logits, non_blocking=True)
        ev[3].record(stream)
        stream.synchronize()
        e2e_marks.append(ev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1), device="cuda")

    # standalone pack / unpack bandwidth, rotating over disjoint block sets so every launch reads cold pages.
    # Timed alone, before the compute-heavy steps pull the clocks down under the power cap: the same condition
    # as the copy measurement the HBM peak comes from (the in-step times are in breakdown_ms_per_step).
    n_sets = max(1, min(8, (pool_blocks - nb_total - 1) // max(nb_suffix, 1)))
    sets_src = [perm_src[nb_total + 1 + i * nb_suffix: nb_total + 1 + (i + 1) * nb_suffix].copy() for i in range(n_sets)]
    sets_dst = [perm_tgt[nb_total + 1 + i * nb_suffix: nb_total + 1 + (i + 1) * nb_suffix].copy() for i in range(n_sets)]
    wires = [torch.empty(wire_elems, dtype=torch.int16, device="cuda") for _ in range(n_sets)]
    payload = wire_elems * 2

    def pack_all():
        for i in range(n_sets):
            kv.kv_pack_blocks(src, sets_src[i], wires[i])

    def unpack_all():
        for i in range(n_sets):
            kv.kv_unpack_assemble(tgt, wires[i], logical, sets_dst[i], tgt_prefix, n, epoch=1, expected_epoch=1)
    pack_all(); unpack_all()
    torch.cuda.synchronize()

    def graph_time(fn, reps=10):
        """Device time per launch with the launches replayed from a CUDA graph, so that host-side call
        overhead (longer than a ~45 us kernel) does not sit between consecutive launches."""
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            g.replay()
            return timed(g.replay, reps) / (reps * n_sets), "cuda-graph replay"
        except Exception:
            return timed(fn, reps) / (reps * n_sets), "direct launches"
    pack_ms, pack_how = graph_time(pack_all)
    unpack_ms, _ = graph_time(unpack_all)
    # the same launches issued directly (no graph): what the gaps between short launches cost by themselves
    pack_direct_ms = timed(pack_all, 10) / (10 * n_sets)
    unpack_direct_ms = timed(unpack_all, 10) / (10 * n_sets)

    # the decode step timed alone as well (direct launches), before the prefill pulls the clocks down
    merged0 = kv.kv_unpack_assemble(tgt, wire, logical, dst_ids, tgt_prefix, n, epoch=1, expected_epoch=1)
    table0 = list(merged0) + extra

    def decode_only():
        kv.kv_decode_step(model, tgt, int(ids[n]), n, table0, logits, workspace=ws_d)
    for _ in range(3):
        decode_only()
    decode_alone_ms = timed(decode_only, 10) / 10

    for _ in range(max(args.warmup, 3)):
        step()
    kv.kv_check_device_status(ws_p)
    kv.kv_check_device_status(ws_d)
    torch.cuda.synchronize()
    kv.kv_profile_read()

    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]) if
                           os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank].isdigit() else local_rank)
    sampler.start()
    kv.kv_profile_enable(True)
    launches0 = kv.kv_launch_count()
    total_ms = timed(step, args.steps)
    launches = kv.kv_launch_count() - launches0
    kv.kv_profile_enable(False)
    prof = kv.kv_profile_read()
    clocks = sampler.stop()
    kv.kv_check_device_status(ws_p)
    kv.kv_check_device_status(ws_d)

    step_e2e()
    e2e_marks.clear()
    e2e_ms = timed(step_e2e, args.steps)
    legs = np.array([[ev[0].elapsed_time(ev[1]), ev[4].elapsed_time(ev[5]), ev[1].elapsed_time(ev[2]),
                      ev[2].elapsed_time(ev[3])] for ev in e2e_marks]).mean(axis=0)

    # prefix-length sweep of the same shape (K/V-only prefill, 3 timed calls each after one warm-up call; then the
    # resumed decode step at that length, 5 timed calls after eight warm-up calls)
    sweep = {}
    if args.sweep and shape_name == "32b" and not args.layers:
        for length in (512, 2048, 8192, 16384):
            table = perm_tgt[: length // bs].copy()
            ids_l = synth.token_ids(shape, seed + 7, length)
            ws_l = model.workspace(kv.KV_OP_PREFILL, length)
            kv.kv_prefill_prefix(model, tgt, ids_l, table, workspace=ws_l)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(3):
                kv.kv_prefill_prefix(model, tgt, ids_l, table, workspace=ws_l)
            e1.record(stream)
            torch.cuda.synchronize()
            kv.kv_check_device_status(ws_l)
            ms = e0.elapsed_time(e1) / 3
            fl = prefill_flops(shape, length)
            sweep[str(length)] = {"ms_per_prefix": round(ms, 3), "tokens_per_s": round(length / (ms * 1e-3), 1),
                                  "tflops": round(fl / (ms * 1e-3) / 1e12, 1),
                                  "bar_ms_60pct_of_burst": round(fl / (0.6 * peaks()["bf16_tflops"] * 1e12) * 1e3, 1)}
            # the resumed decode step at this length's resume position n = prefix + prefix / 8 (the suffix pages hold
            # whatever finite K/V earlier runs left there: the step's cost does not depend on the values)
            n_l = length + length // 8
            table_d = perm_tgt[: n_l // bs + 1].copy()
            ws_dl = model.workspace(kv.KV_OP_DECODE, n_l + 1)
            for _ in range(8):      # long enough for the memory system to recover from the power-capped prefill
                kv.kv_decode_step(model, tgt, int(ids_l[0]), n_l, table_d, logits, workspace=ws_dl)
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(5):
                kv.kv_decode_step(model, tgt, int(ids_l[0]), n_l, table_d, logits, workspace=ws_dl)
            e1.record(stream)
            torch.cuda.synchronize()
            sweep[str(length)]["decode_step_ms_at_resume"] = round(e0.elapsed_time(e1) / 5, 3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    pk = peaks()
    ms_per_step = total_ms / args.steps
    value = replicas.whole_job_throughput(prefix, world, ms_per_step)
    per_step = {k: (ms / args.steps, cnt // args.steps) for k, (ms, cnt) in prof.items()}
    prefill_kinds = ("embed", "rmsnorm", "gemm_qkv", "rope_store", "attention", "gemm_o", "gemm_gate_up", "gemm_down")
    prefill_ms = sum(per_step[k][0] for k in prefill_kinds)
    decode_ms = sum(per_step[k][0] for k in ("decode_gemv", "decode_attention", "decode_other", "lm_head"))
    gu_ms, gu_launches = prof["gemm_gate_up"]
    gu_flops = 2.0 * prefix * shape.hidden * 2 * shape.ffn
    achieved = gu_flops / (gu_ms / max(gu_launches, 1) * 1e-3) / 1e12 if gu_ms > 0 else 0.0
    flops = prefill_flops(shape, prefix)
    sm_mhz = clocks.get("sm_mhz") or 0.0
    hw_peak = hw_tensor_peak_tflops(sm_mhz) if sm_mhz else None
    traffic = NCU_TRAFFIC_BYTES.get(args.workload) if not args.layers else None
    roofline = {"bound": "tensor", "kernel": "gemm_tc_pair_kernel<SWIGLU, 256> (gate/up projection, cta_group::2)", "achieved": achieved,
                "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": achieved / pk["bf16_tflops_sustained"],
                "peak_source": pk["source"] + " library bf16 matmul, sustained (the kernel is timed inside a long power-capped step)",
                "frac_of_burst_peak": achieved / pk["bf16_tflops"],
                "tensor_pipe_peak_at_sampled_clock": hw_peak,
                "frac_of_tensor_pipe_at_sampled_clock": achieved / hw_peak if hw_peak else None,
                "tensor_pipe_model": f"{SM_COUNT} SMs x {BF16_FLOP_PER_CLK_PER_SM} bf16 flop/clk/SM x median sampled SM clock",
                "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                "flops_per_launch": gu_flops, "launches_timed": gu_launches,
                "traffic": traffic,
                "traffic_source": ("ncu capture summarised in profiles/gemm_tc_pair_gate_up_32b-4k.md (same shape, one launch); "
                                   "not measured in this run") if traffic else None}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(args.workload, world=world, layers=args.layers),
        "clocks": clocks,
        "e2e": {"value": world * prefix / (e2e_ms / args.steps * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": int(payload + 4 * (prefix + nb_prefix + nb_total + 1 + nb_suffix * 2)),
                "d2h_bytes_per_step": int(payload + 4 * shape.vocab), "ms_per_step": e2e_ms / args.steps,
                "prefill_ms": float(legs[0]), "copy_ms": float(legs[1] + legs[3]),
                "pack_wire_d2h_h2d_ms": float(legs[1]), "logits_d2h_ms": float(legs[3]),
                "unpack_decode_ms": float(legs[2]),
                "note": "legs are CUDA-event times inside the end-to-end step (mean over the timed steps); pack and the "
                        "wire's device-to-host and host-to-device copies run on a side stream beside the prefill (the "
                        "method's parallel preparation), assembly waits for both"},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "prefill": {"ms_per_prefix": prefill_ms, "tokens_per_s": prefix / (prefill_ms * 1e-3),
                    "tflops": flops / (prefill_ms * 1e-3) / 1e12,
                    "frac_of_bf16_burst_peak": flops / (prefill_ms * 1e-3) / 1e12 / pk["bf16_tflops"],
                    "frac_of_bf16_sustained_peak": flops / (prefill_ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
                    "frac_of_tensor_pipe_at_sampled_clock": flops / (prefill_ms * 1e-3) / 1e12 / hw_peak if hw_peak else None,
                    "frac_of_nominal_2250": flops / (prefill_ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS},
        "pack": {"gbs": 2 * payload / (pack_ms * 1e-3) / 1e9, "frac_of_hbm": 2 * payload / (pack_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                 "us": pack_ms * 1e3, "payload_bytes": payload,
                 "timing": f"{pack_how} of {n_sets} launches over disjoint block sets",
                 "direct_launch_us": pack_direct_ms * 1e3,
                 "in_step_us": per_step["pack"][0] * 1e3,
                 "frac_in_step": 2 * payload / (per_step["pack"][0] * 1e-3) / 1e9 / pk["hbm_gbs"],
                 "in_step_note": "CUDA events around the one launch, right behind the power-capped prefill"},
        "unpack": {"gbs": 2 * payload / (unpack_ms * 1e-3) / 1e9,
                   "frac_of_hbm": 2 * payload / (unpack_ms * 1e-3) / 1e9 / pk["hbm_gbs"], "us": unpack_ms * 1e3,
                   "direct_launch_us": unpack_direct_ms * 1e3,
                   "in_step_us": per_step["unpack"][0] * 1e3,
                   "frac_in_step": 2 * payload / (per_step["unpack"][0] * 1e-3) / 1e9 / pk["hbm_gbs"]},
        "decode_step_ms": decode_ms,
        "decode_step_alone_ms": decode_alone_ms,
        "t0_analog_ms": per_step["unpack"][0] + decode_ms,
        "breakdown_ms_per_step": {k: round(v[0], 4) for k, v in per_step.items()},
    }
    # every kernel class of the step against the measured peak that bounds it (the library matmul's sustained rate
    # for the tensor-bound classes, the copy bandwidth for the HBM-bound ones), from the event times above
    if not args.layers:
        table = {}
        for kind, (amount, unit) in step_work(shape, prefix, suffix).items():
            ms = per_step[kind][0]
            if ms <= 0:
                continue
            if unit == "flop":
                rate = amount / (ms * 1e-3) / 1e12
                table[kind] = {"ms": round(ms, 3), "tflops": round(rate, 1), "frac_of_sustained_peak": round(rate / pk["bf16_tflops_sustained"], 3)}
            else:
                rate = amount / (ms * 1e-3) / 1e9
                table[kind] = {"ms": round(ms, 4), "gbs": round(rate, 1), "frac_of_hbm": round(rate / pk["hbm_gbs"], 3)}
        line["kernel_rooflines_in_step"] = table
    if sweep:
        line["sweep"] = sweep
    # Algorithm 1 fed with the rates measured above (Section 4.2): prefill rate r_p, decode rate r_d of the
    # source (taken as this GPU's decode step), T_0 = assembly + first decode step, on two configured links.
    s_kv = kv.kv_bytes_per_token(shape.n_layers, shape.n_kv_heads, shape.head_dim, 2)
    r_p, r_d = prefix / (prefill_ms * 1e-3), 1.0 / (decode_alone_ms * 1e-3)
    t0 = (unpack_ms + decode_alone_ms) * 1e-3
    line["window"] = {"inputs": {"k_curr": prefix, "r_p": r_p, "r_d": r_d, "s_kv": s_kv, "t0": t0, "alpha": 0.8,
                                 "t_remain": 5.0, "t_max": 5.0, "d_t": 0.01}, "links": {}}
    for name, goodput in (("300 Mbit/s", 300e6 / 8), ("NVLink 770 GB/s", 770e9)):
        best, trig = kv.kv_window_select(5.0, 0.01, k_curr=float(prefix), r_p=r_p, r_d=r_d, goodput=goodput,
                                         s_kv=float(s_kv), t0=t0, t_load=0.0, alpha=0.8, t_remain=5.0)
        line["window"]["links"][name] = {"t_w_star": best["t_w"], "t_sit": best["t_sit"], "t_early": best["t_early"],
                                         "trigger_now": trig}
    if world == 1 and not args.no_cpu_baseline:
        ref_warmup = max(args.ref_warmup, args.warmup if args.warmup_given else 0)
        line["cpu_baseline"] = cpu_baseline(synth.SHAPES[shape_name], prefix,
                                            oracle_sample_tokens(prefix, args.ref_tokens, args.steps, ref_warmup),
                                            suffix_blocks=-(-suffix // synth.SHAPES[shape_name].block_size))
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------------------------------ pack/unpack stress
def stress_geometry(kv, torch, shape):
    """Source pool of 32,768 blocks (128 GiB at the 32B shape) when it fits beside a 5,120-block destination pool
    and the 18.1 GiB of wire buffers; otherwise the source pool is halved until it does (only referenced pages
    are touched, so the pool size changes the address spread, not the bytes moved)."""
    counts = list(synth.STRESS_BLOCK_COUNTS)
    total = sum(counts)
    page = synth.kv_page_bytes(shape)
    block_bytes = 2 * shape.n_layers * page
    dst_blocks = 5120
    free, _ = torch.cuda.mem_get_info()
    src_blocks = 32768
    while src_blocks > total and (src_blocks + dst_blocks + total) * block_bytes + (2 << 30) > free:
        src_blocks //= 2
    return counts, total, src_blocks, dst_blocks, block_bytes


def run_stream_overlap(args):
    """Source-side incremental suffix synchronisation (Section 4.3): decode steps of the 32B shape with every completed
    suffix block packed on a side stream and delivered to a receiver on the same GPU, against the same steps alone."""
    import torch
    import paper_2608_16477_b200 as kv
    from paper_2608_16477_b200 import streaming
    kv.load()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    shape = synth.SHAPES["32b"]
    k_split, n_steps = 4096, 64
    bs = shape.block_size
    nb = (k_split + n_steps) // bs + 1
    model, _ = build_model(kv, torch, shape)
    src = kv.PagedCache(shape, nb + 8)
    tgt = kv.PagedCache(shape, nb + 8)
    kv.kv_fill_pattern(src.data, src.data.numel() * 2, seed=5)
    src.data.bitwise_and_(0x3FFF)                      # finite bf16 content standing in for the prefix K/V
    table = synth.block_permutation(1, nb + 8)[:nb]
    ids = synth.token_ids(shape, 0, k_split + n_steps + 1)
    logits = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    ws = model.workspace(kv.KV_OP_DECODE, k_split + n_steps + 1)
    stream = torch.cuda.current_stream()

    def decode_run(streamer):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for pos in range(k_split, k_split + n_steps):
            kv.kv_decode_step(model, src, int(ids[pos]), pos, table[: pos // bs + 1], logits, workspace=ws)
            if streamer is not None:
                streamer.on_token(pos)
                streamer.pump()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n_steps

    for _ in range(max(args.warmup, 3)):
        decode_run(None)
    plain = min(decode_run(None) for _ in range(args.steps))
    times, sent = [], 0
    for rep in range(args.steps):
        rx = streaming.SuffixReceiver(tgt, 1, rep, k_split, n_steps // bs + 1, list(range(nb + 8))[-(n_steps // bs + 1):])
        st = streaming.SuffixStreamer(src, table, k_split, 1, rep, streaming.LoopbackTransport(rx))
        times.append(decode_run(st))
        sent = len(st.sent)
    overlapped = min(times)
    block_bytes = shape.n_layers * 2 * src.page_bytes
    line = {"metric": "decode_ms_with_suffix_streaming", "value": overlapped, "unit": "ms", "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": overlapped, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "stream-overlap", "shape": "32b", "k_split": k_split, "decode_steps": n_steps,
                       "blocks_streamed": sent, "block_bytes": block_bytes},
            "decode_ms_alone": plain, "decode_ms_streaming": overlapped, "slowdown": overlapped / plain - 1.0,
            "gpu_launches": int(kv.kv_launch_count())}
    print(json.dumps(line))
    return 0


def run_batched_prefill(args):
    """Concurrent migrations (Section 4.5): 4 prefixes per GPU rebuilt by one kv_prefill_prefix_batched call against
    separate kv_prefill_prefix calls, 32B shape.  With N GPUs the 4 N independent requests are dealt out over the ranks
    (replicas.requests_of_rank), each rank rebuilds its share, no data-path collective."""
    import torch
    import torch.distributed as dist
    import paper_2608_16477_b200 as kv
    from paper_2608_16477_b200 import replicas
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    kv.load()
    shape = synth.SHAPES["32b"]
    n = 512
    mine = replicas.requests_of_rank(4 * world, world, rank)
    k_req = len(mine)
    model, _ = build_model(kv, torch, shape, 1000 + rank)
    blocks_each = n // shape.block_size
    cache = kv.PagedCache(shape, k_req * blocks_each + 8, fill=0)
    perm = synth.block_permutation(3, k_req * blocks_each + 8)
    ids = [synth.token_ids(shape, 10 + r, n) for r in mine]
    tabs = [perm[i * blocks_each:(i + 1) * blocks_each].copy() for i in range(k_req)]

    def separate():
        for i in range(k_req):
            kv.kv_prefill_prefix(model, cache, ids[i], tabs[i])

    def batched():
        kv.kv_prefill_prefix_batched(model, cache, ids, tabs)

    def timed(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return replicas.max_over_ranks(e0.elapsed_time(e1) / args.steps, device="cuda")
    ms_sep, ms_bat = timed(separate), timed(batched)
    if rank == 0:
        line = {"metric": METRIC, "value": replicas.whole_job_throughput(k_req * n, world, ms_bat), "unit": UNIT,
                "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_bat, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "batched-prefill", "shape": "32b", "requests_per_gpu": k_req, "prefix_tokens": n,
                           "parallelism": f"replicas x{world}: requests dealt out round-robin over the ranks"},
                "batched_ms": ms_bat, "separate_calls_ms": ms_sep,
                "separate_calls_tokens_per_s": replicas.whole_job_throughput(k_req * n, world, ms_sep),
                "gpu_launches": int(kv.kv_launch_count())}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_chunk_interleave(args):
    """Contention-aware migration (Section 4.5): the target keeps serving a resident request while it rebuilds a
    migrating request's 4,096-token prefix in chunks, one resident decode step after every chunk, on one stream.
    Reports, for 256-token chunks (the chunk size of Section 6.3) and 1,024-token chunks, what the resident request
    sees (time between its tokens while the migration runs, against its undisturbed decode step) and what the
    migration pays (chunked and interleaved rebuild against one uninterrupted prefill call), 32B shape."""
    import torch
    import paper_2608_16477_b200 as kv
    kv.load()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    shape = synth.SHAPES["32b"]
    prefix, resident_ctx, chunk_sizes = 4096, 2048, (256, 1024)
    bs = shape.block_size
    max_steps = prefix // min(chunk_sizes)
    res_blocks = (resident_ctx + max_steps) // bs + 1
    mig_blocks = prefix // bs
    model, _ = build_model(kv, torch, shape)
    cache = kv.PagedCache(shape, res_blocks + mig_blocks + 8)
    kv.kv_fill_pattern(cache.data, cache.data.numel() * 2, seed=5)
    cache.data.bitwise_and_(0x3FFF)                    # finite bf16 content standing in for the resident request's K/V
    perm = synth.block_permutation(1, res_blocks + mig_blocks + 8)
    res_table, mig_table = perm[:res_blocks], perm[res_blocks:res_blocks + mig_blocks]
    res_ids = synth.token_ids(shape, 0, resident_ctx + max_steps + 1)
    mig_ids = synth.token_ids(shape, 1, prefix)
    logits = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    ws_d = model.workspace(kv.KV_OP_DECODE, resident_ctx + max_steps + 1)
    ws_p = model.workspace(kv.KV_OP_PREFILL, prefix)
    stream = torch.cuda.current_stream()

    def decode(i):
        pos = resident_ctx + i
        kv.kv_decode_step(model, cache, int(res_ids[pos]), pos, res_table[: pos // bs + 1], logits, workspace=ws_d)

    def prefill_chunk(c, chunk):
        kv.kv_prefill_prefix(model, cache, mig_ids[c * chunk:(c + 1) * chunk], mig_table[: (c + 1) * chunk // bs],
                             pos0=c * chunk, workspace=ws_p)

    def measure(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        best = None
        for _ in range(args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
        return best

    def decode_alone():
        for i in range(max_steps):
            decode(i)

    def chunked(chunk, with_decode):
        def run():
            for c in range(prefix // chunk):
                prefill_chunk(c, chunk)
                if with_decode:
                    decode(c)
        return run

    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    l0 = kv.kv_launch_count()
    itl_alone = measure(decode_alone) / max_steps
    one_call = measure(lambda: kv.kv_prefill_prefix(model, cache, mig_ids, mig_table, workspace=ws_p))
    per_chunk = {}
    for chunk in chunk_sizes:
        alone, busy = measure(chunked(chunk, False)), measure(chunked(chunk, True))
        itl = busy / (prefix // chunk)
        per_chunk[str(chunk)] = {"rebuild_ms": alone, "rebuild_ms_with_resident_decode": busy,
                                 "rebuild_vs_one_call": alone / one_call, "resident_ms_between_tokens": itl,
                                 "resident_slowdown": itl / itl_alone}
    launches = kv.kv_launch_count() - l0
    clocks = sampler.stop()
    kv.kv_check_device_status(ws_p)
    head = per_chunk[str(chunk_sizes[0])]
    line = {"metric": METRIC, "value": prefix / (head["rebuild_ms_with_resident_decode"] * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": head["rebuild_ms_with_resident_decode"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "chunk-interleave", "shape": "32b", "prefix_tokens": prefix,
                       "chunk_tokens": list(chunk_sizes), "resident_context": resident_ctx,
                       "l2": "weights (62 GB per pass) larger than L2"},
            "rebuild_ms_one_call": one_call, "resident_ms_between_tokens_alone": itl_alone, "chunks": per_chunk,
            "clocks": clocks, "gpu_launches": int(launches)}
    print(json.dumps(line))
    return 0


def run_pack_stress(args):
    import torch
    import paper_2608_16477_b200 as kv
    kv.load()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    shape = synth.SHAPES["32b"]
    counts, total, src_blocks, dst_blocks, block_bytes = stress_geometry(kv, torch, shape)
    src = kv.PagedCache(shape, src_blocks)
    dst = kv.PagedCache(shape, dst_blocks, fill=0)
    kv.kv_fill_pattern(src.data, src.data.numel() * 2, seed=77)
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    src_ids = synth.block_permutation(1, src_blocks)[:total]
    dst_ids = synth.block_permutation(2, dst_blocks)[:total]
    wires = [torch.empty(c * block_bytes, dtype=torch.uint8, device="cuda") for c in counts]
    stream = torch.cuda.current_stream()

    def timed(fn, reps):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    pack = lambda: kv.kv_pack_blocks_batched(src, offs, src_ids, wires)
    unpack = lambda: kv.kv_unpack_blocks_batched(dst, offs, dst_ids, wires)
    for _ in range(max(args.warmup, 3)):
        pack(); unpack()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    l0 = kv.kv_launch_count()
    pack_ms = timed(pack, args.steps)
    unpack_ms = timed(unpack, args.steps)
    launches = kv.kv_launch_count() - l0
    clocks = sampler.stop()
    kv.kv_check_copy_status()
    pk = peaks()
    payload = total * block_bytes
    gbs = lambda ms: 2 * payload / (ms * 1e-3) / 1e9
    line = {"metric": "kv_pack_unpack_gbs", "value": gbs(pack_ms), "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": pack_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": "pack-stress", "requests": len(counts), "blocks": total, "payload_bytes": payload,
                       "src_pool_blocks": src_blocks, "dst_pool_blocks": dst_blocks,
                       "l2": "inputs larger than L2 (18.1 GiB payload per launch set)"},
            "clocks": clocks, "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": "copy_pages_kernel", "achieved": gbs(pack_ms), "peak": pk["hbm_gbs"],
                         "unit": "GB/s", "frac": gbs(pack_ms) / pk["hbm_gbs"], "peak_source": pk["source"], "traffic": None},
            "pack": {"gbs": gbs(pack_ms), "ms": pack_ms, "frac_of_hbm": gbs(pack_ms) / pk["hbm_gbs"]},
            "unpack": {"gbs": gbs(unpack_ms), "ms": unpack_ms, "frac_of_hbm": gbs(unpack_ms) / pk["hbm_gbs"]}}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="32b-4k", choices=sorted(WORKLOADS) + ["pack-stress", "stream-overlap", "batched-prefill", "chunk-interleave"])
    ap.add_argument("--layers", type=int, default=0, help="debug: reduced depth (invalid as a bench number)")
    ap.add_argument("--ref-tokens", type=int, default=4096, help="prefix tokens in the oracle's bounded sample")
    ap.add_argument("--ref-warmup", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", dest="sweep", action="store_false",
                    help="skip the prefix-length sweep (512 / 2,048 / 8,192 / 16,384 tokens) after the timed region")
    args = ap.parse_args()
    args.warmup_given = any(a == "--warmup" or a.startswith("--warmup=") for a in sys.argv[1:])
    if args.workload == "pack-stress" and args.impl != "reference":
        return run_pack_stress(args)
    if args.workload == "stream-overlap" and args.impl != "reference":
        return run_stream_overlap(args)
    if args.workload == "batched-prefill" and args.impl != "reference":
        return run_batched_prefill(args)
    if args.workload == "chunk-interleave" and args.impl != "reference":
        return run_chunk_interleave(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
