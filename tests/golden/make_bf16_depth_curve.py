#!/usr/bin/env python
"""Writes tests/golden/bf16_depth_curve_8b.txt: how far two-byte storage of activations and of the cache
moves the K/V of a deep decoder away from the exact definition, layer by layer.  Calls only oracle/ and the
seeded input generators (synth/); no GPU, no CUDA library.

  python tests/golden/make_bf16_depth_curve.py [--tokens 256] [--layers 36] [--out FILE]

Three evaluations of the same prefill (8B-shaped decoder, N(0, 0.02) weights, norm gains 1, token ids uniform
over the vocabulary) advance in lockstep so each layer's weights are generated once:
  exact   the definition, fp64 throughout;
  bf16    the same function with every tensor that sits between two contractions of a 16-bit pipeline held in
          bfloat16 (normed activations, post-RoPE Q and K, V, attention output, SwiGLU output), arithmetic
          still fp64: what ANY pipeline with a two-byte cache and two-byte tensor-core operands computes at best;
  bf16/32 as bf16, with the matrix products accumulated in fp32 by the library instead of fp64: a second
          realisation of the same roundings whose only difference is summation order and precision.
Columns: layer, rel-L2(K bf16 vs exact), rel-L2(V bf16 vs exact), rel-L2(K bf16/32 vs bf16), rel-L2(V bf16/32 vs
bf16).  The first pair is the floor below which no two-byte pipeline can stay; the second pair is the distance
between two correct realisations of that pipeline (rounding decisions flip when the pre-rounding values differ
in the last bits, and later layers amplify the flips).
"""
import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402
from oracle import kv_oracle as O  # noqa: E402

DEFAULT_OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "bf16_depth_curve_8b.txt")
SEED = 0
VOCAB = 8192     # the LM head plays no part in K/V; a small table keeps the embedding draw cheap


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.sqrt(np.sum((a - b) ** 2) / np.sum(b ** 2)))


def curve(shape, n_tokens, n_layers, seed=SEED, log=None):
    """Rows (layer, eK, eV, dK, dV) for the first n_layers layers."""
    ids = synth.token_ids(shape, seed, n_tokens)
    head = synth.head_weights(shape, seed)
    x0 = np.asarray(head["embed"], dtype=np.float64)[ids]
    pos = np.arange(n_tokens)
    xe, xb, xc = x0, x0, x0
    rows = []
    for l in range(n_layers):
        t0 = time.time()
        w = synth.layer_weights(shape, seed, l)
        xe, ke, ve = O.layer_forward(shape, w, xe, pos)
        xb, kb, vb = O.layer_forward(shape, w, xb, pos, act_bf16=True)
        xc, kc, vc = O.layer_forward(shape, w, xc, pos, act_bf16=True, mm_dtype=np.float32)
        rows.append((l, rel_l2(kb, ke), rel_l2(vb, ve), rel_l2(kc, kb), rel_l2(vc, vb)))
        if log is not None:
            log(f"layer {l}: " + " ".join(f"{v:.4e}" for v in rows[-1][1:]) + f"  ({time.time() - t0:.1f} s)")
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=256)
    ap.add_argument("--layers", type=int, default=0, help="0: the shape's full depth")
    ap.add_argument("--out", default=DEFAULT_OUT)
    args = ap.parse_args()
    shape = synth.ModelShape(**{**synth.SHAPES["8b"].__dict__, "vocab": VOCAB})
    n_layers = args.layers or shape.n_layers
    rows = curve(shape, args.tokens, n_layers, log=lambda s: print(s, file=sys.stderr, flush=True))
    with open(args.out, "w") as f:
        f.write("# Distance between the exact K/V and the K/V of the same decoder evaluated with bfloat16 storage points,\n"
                "# per layer; written by tests/golden/make_bf16_depth_curve.py from the CPU oracle alone.\n"
                f"# shape 8b (hidden 4096, 32 Q / 8 KV heads of 128, FFN 12288), vocab {VOCAB}, seed {SEED}, "
                f"{args.tokens} tokens\n"
                "# layer  relL2_K(bf16 vs exact)  relL2_V(bf16 vs exact)  relL2_K(bf16 fp32-mm vs bf16)  relL2_V(same)\n")
        for r in rows:
            f.write(f"{r[0]:d} {r[1]:.4e} {r[2]:.4e} {r[3]:.4e} {r[4]:.4e}\n")
    print(args.out)


if __name__ == "__main__":
    main()
