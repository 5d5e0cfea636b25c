"""Runs ONE kernel of the hot path a few times at the benchmark's shapes, for profiler captures.

  python profile_case.py gemm_gate_up [--tokens 4096] [--iters 3]
  cases: gemm_qkv, gemm_o, gemm_gate_up, gemm_down, attention, rmsnorm, pack, unpack, pack_batched, unpack_batched,
         decode_gemv (gate/up), decode_gemv_o, decode_gemv_down, decode_gemv_qkv, decode_gemv_lm_head, decode_attention,
         prefill_layer

Inputs are synthetic and larger than L2 where the kernel is bandwidth-bound; a few GB at most are held on
the device so a multi-pass capture stays short.  Prints the CUDA-event time per launch.
"""
import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402


def main():
    import torch
    import paper_2608_16477_b200 as kv
    ap = argparse.ArgumentParser()
    ap.add_argument("case")
    ap.add_argument("--shape", default="32b")
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--blocks", type=int, default=32, help="pack/unpack: blocks per launch")
    ap.add_argument("--pair", action="store_true", help="GEMM cases: the CTA-pair (cta_group::2) kernel")
    a = ap.parse_args()
    kv.load()
    s = synth.SHAPES[a.shape]
    t = a.tokens
    dev = "cuda"
    g = torch.Generator(device=dev).manual_seed(0)

    def rnd(*shape, std=1.0):
        return torch.empty(*shape, dtype=torch.bfloat16, device=dev).normal_(0.0, std, generator=g)
    status = torch.zeros(64, dtype=torch.int32, device=dev)
    if a.case.startswith("gemm"):
        if a.case == "gemm_gate_up":
            x, w, mode = rnd(t, s.hidden), rnd(2 * s.ffn, s.hidden, std=0.02), 2
            out, resid, flops = torch.empty(t, s.ffn, dtype=torch.bfloat16, device=dev), None, 2.0 * t * s.hidden * 2 * s.ffn
        elif a.case == "gemm_down":
            x, w, mode = rnd(t, s.ffn), rnd(s.hidden, s.ffn, std=0.02), 1
            out, resid, flops = None, torch.zeros(t, s.hidden, dtype=torch.float32, device=dev), 2.0 * t * s.hidden * s.ffn
        elif a.case == "gemm_o":
            x, w, mode = rnd(t, s.q_dim), rnd(s.hidden, s.q_dim, std=0.02), 1
            out, resid, flops = None, torch.zeros(t, s.hidden, dtype=torch.float32, device=dev), 2.0 * t * s.hidden * s.q_dim
        elif a.case == "gemm_o_store":          # the O-projection's shape with the plain bf16-store epilogue
            x, w, mode = rnd(t, s.q_dim), rnd(s.hidden, s.q_dim, std=0.02), 0
            out, resid, flops = torch.empty(t, s.hidden, dtype=torch.bfloat16, device=dev), None, 2.0 * t * s.hidden * s.q_dim
        elif a.case == "gemm_qkv":
            x, w, mode = rnd(t, s.hidden), rnd(s.qkv_dim, s.hidden, std=0.02), 0
            out, resid, flops = torch.empty(t, s.qkv_dim, dtype=torch.bfloat16, device=dev), None, 2.0 * t * s.hidden * s.qkv_dim
        else:
            raise SystemExit(f"unknown case {a.case}")
        flag = 0x100 if a.pair else 0     # KV_GEMM_CTA_PAIR
        run = lambda: kv.kv_op_gemm(x, w, mode | flag, out=out, resid=resid, status=status)
        work, unit = flops / 1e12, "TFLOP/s"
    elif a.case == "attention":
        qkv = rnd(t, s.qkv_dim)
        out = torch.empty(t, s.q_dim, dtype=torch.bfloat16, device=dev)
        run = lambda: kv.kv_op_attention_prefill(qkv, s.n_q_heads, s.n_kv_heads, s.head_dim, out, status=status)
        work, unit = 2.0 * s.n_q_heads * s.head_dim * t * (t + 1) / 1e12, "TFLOP/s"
    elif a.case in ("pack", "unpack"):
        pool = 1024                                   # 4 GiB pool at the 32B shape
        cache = kv.PagedCache(s, pool)
        kv.kv_fill_pattern(cache.data, cache.data.numel() * 2, seed=1)
        perm = synth.block_permutation(1, pool)
        n_sets = 4
        wires = [torch.empty(a.blocks * s.n_layers * 2 * cache.page_bytes, dtype=torch.uint8, device=dev)
                 for _ in range(n_sets)]
        state = {"i": 0}

        def run():
            i = state["i"] % n_sets
            state["i"] += 1
            ids = perm[i * a.blocks:(i + 1) * a.blocks]
            if a.case == "pack":
                kv.kv_pack_blocks(cache, ids, wires[i])
            else:
                kv.kv_unpack_assemble(cache, wires[i], np.arange(a.blocks), ids, [], a.blocks * s.block_size)
        work, unit = 2.0 * a.blocks * s.n_layers * 2 * cache.page_bytes / 1e9, "GB/s"
    elif a.case in ("pack_batched", "unpack_batched"):
        # the 16-request stress workload at 1/16 of its block counts (289 blocks, 1.1 GiB payload) in the batched form:
        # one launch for all requests
        pool = 1024
        cache = kv.PagedCache(s, pool)
        kv.kv_fill_pattern(cache.data, cache.data.numel() * 2, seed=1)
        counts = [max(1, c // 16) for c in synth.STRESS_BLOCK_COUNTS]
        offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        n_sets = 2
        perms = [synth.block_permutation(1 + i, pool)[: offs[-1]] for i in range(n_sets)]
        block_bytes = s.n_layers * 2 * cache.page_bytes
        wires = [[torch.empty(c * block_bytes, dtype=torch.uint8, device=dev) for c in counts] for _ in range(n_sets)]
        state = {"i": 0}

        def run():
            i = state["i"] % n_sets
            state["i"] += 1
            if a.case == "pack_batched":
                kv.kv_pack_blocks_batched(cache, offs, perms[i], wires[i])
            else:
                kv.kv_unpack_blocks_batched(cache, offs, perms[i], wires[i])
        work, unit = 2.0 * int(offs[-1]) * block_bytes / 1e9, "GB/s"
    elif a.case in ("decode_gemv_o", "decode_gemv_down", "decode_gemv_qkv", "decode_gemv_lm_head"):
        # the other products of one decode step, each as its own (SHORT) launch, rotating over enough weight copies to
        # exceed L2: O projection 5120 x 8192 (84 MB, residual add), down projection 5120 x 25600 (262 MB, residual add),
        # a QKV-sized product 10240 x 5120 (105 MB, norm folded in), the LM head 151936 x 5120 (1.56 GB, norm folded in)
        rows, k, mode, norm = {"decode_gemv_o": (s.hidden, s.q_dim, 1, False), "decode_gemv_down": (s.hidden, s.ffn, 1, False),
                               "decode_gemv_qkv": (s.qkv_dim, s.hidden, 0, True),
                               "decode_gemv_lm_head": (s.vocab, s.hidden, 0, True)}[a.case]
        copies = max(2, int(400e6 // (rows * k * 2)) + 1)
        ws = [rnd(rows, k, std=0.02) for _ in range(copies)]
        x = torch.randn(k, device=dev)
        gain = torch.ones(k, dtype=torch.bfloat16, device=dev) if norm else None
        y = torch.zeros(rows, device=dev)
        state = {"i": 0}

        def run():
            state["i"] += 1
            kv.kv_op_gemv(ws[state["i"] % copies], x, mode, y, gain=gain, eps=1e-6)
        work, unit = ws[0].numel() * 2 / 1e9, "GB/s"
    elif a.case == "rmsnorm":
        # one normalisation pass of the prefill: tokens x hidden fp32 -> bf16, rotating over four inputs (> L2)
        xs = [torch.randn(t, s.hidden, device=dev) for _ in range(4)]
        gain = torch.ones(s.hidden, dtype=torch.bfloat16, device=dev)
        outs = [torch.empty(t, s.hidden, dtype=torch.bfloat16, device=dev) for _ in range(4)]
        state = {"i": 0}

        def run():
            state["i"] += 1
            kv.kv_op_rmsnorm(xs[state["i"] % 4], gain, 1e-6, outs[state["i"] % 4])
        work, unit = t * s.hidden * 6 / 1e9, "GB/s"
    elif a.case == "decode_gemv":
        # the gate/up product of one decode step (524 MB of weights), rotating over 4 weight copies (> L2)
        ws = [rnd(2 * s.ffn, s.hidden, std=0.02) for _ in range(4)]
        x = torch.randn(s.hidden, device=dev)
        gain = torch.ones(s.hidden, dtype=torch.bfloat16, device=dev)
        y = torch.empty(s.ffn, device=dev)
        state = {"i": 0}

        def run():
            state["i"] += 1
            kv.kv_op_gemv(ws[state["i"] % 4], x, 2, y, gain=gain, eps=1e-6)
        work, unit = ws[0].numel() * 2 / 1e9, "GB/s"
    elif a.case == "prefill_layer":
        # one decoder layer of the shape through kv_prefill_prefix (logits on, so the layer is not truncated after
        # its QKV projection): the way to capture the QKV + RoPE + paged-store GEMM, whose epilogue needs a cache
        s1 = s.with_layers(1)
        mat = lambda r, c: rnd(r, c, std=0.02)
        ones = lambda: torch.ones(s.hidden, dtype=torch.bfloat16, device=dev)
        layer = lambda l: {"attn_norm": ones(), "ffn_norm": ones(), "w_qkv": mat(s.qkv_dim, s.hidden),
                           "w_o": mat(s.hidden, s.q_dim), "w_gate_up": mat(2 * s.ffn, s.hidden), "w_down": mat(s.hidden, s.ffn)}
        head = {"embed": mat(s.vocab, s.hidden), "lm_head": mat(s.vocab, s.hidden), "final_norm": ones()}
        model = kv.Model(s1, head, layer)
        cache = kv.PagedCache(s1, t // s.block_size + 1)
        ids = synth.token_ids(s1, 0, t)
        table = synth.block_permutation(1, t // s.block_size + 1)[: t // s.block_size]
        ws = model.workspace(kv.KV_OP_PREFILL, t)
        logits = torch.empty(s.vocab, dtype=torch.float32, device=dev)
        run = lambda: kv.kv_prefill_prefix(model, cache, ids, table, logits_out=logits, workspace=ws)
        lin = 2.0 * t * (s.hidden * s.qkv_dim + s.q_dim * s.hidden + 3 * s.hidden * s.ffn)
        work, unit = (lin + 2.0 * s.n_q_heads * s.head_dim * t * (t + 1)) / 1e12, "TFLOP/s"
    elif a.case == "decode_attention":
        # one layer's paged attention of a decode step at context a.tokens + 512 (the bench's resume position),
        # rotating over 4 layers of a fragmented cache so consecutive launches read cold pages
        n_ctx = t + 512 + 1
        pool = 1024
        layers = 4
        s4 = s.with_layers(layers)
        cache = kv.PagedCache(s4, pool)
        kv.kv_fill_pattern(cache.data, cache.data.numel() * 2, seed=1)
        cache.data.bitwise_and_(0x3FFF)               # small finite bf16 values
        table = torch.from_numpy(np.ascontiguousarray(synth.block_permutation(2, pool)[: -(-n_ctx // s.block_size)]
                                                      .astype(np.int32))).to(dev)
        q = torch.randn(s.n_q_heads, s.head_dim, device=dev)
        out = torch.empty(s.n_q_heads, s.head_dim, device=dev)
        scratch = torch.empty(kv.kv_paged_attention_scratch_bytes(s.n_q_heads, s.head_dim, n_ctx), dtype=torch.uint8, device=dev)
        state = {"i": 0}

        def run():
            state["i"] += 1
            kv.kv_op_paged_attention(q, cache, state["i"] % layers, table, n_ctx, scratch, out)
        work, unit = 2.0 * n_ctx * s.n_kv_heads * s.head_dim * 2 / 1e9, "GB/s"
    else:
        raise SystemExit(f"unknown case {a.case}")
    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    if int(status[0]) != 0:
        raise SystemExit(f"device wait ran out: {status[:8].tolist()}")
    per = work / (ms * 1e-3)
    print(f"{a.case}: {ms * 1e3:.1f} us per launch, {per:.1f} {unit}")
    return 0


if __name__ == "__main__":
    sys.exit(main())
