"""Shared driver of the end-to-end parity scenario (test helper; imports both the oracle and the binding).

tokens t[0..n] (n+1 ids, teacher-forced): the source cache is built by prefill(t[0:k]) followed by decode
steps for t[k..n-1]; the target cache by prefill(t[0:k]) into its own fresh blocks; the suffix blocks are
packed at the source, unpacked/assembled at the target, and the target resumes with decode_step(t[n], pos=n).
Reference values: the oracle's full forward over t[0..n].
"""
import os

import numpy as np

import synth
from oracle import kv_oracle as O

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def depth_curve():
    """Per-layer distances written by tests/golden/make_bf16_depth_curve.py from the oracle alone:
    e[l] = relative L2 between the exact K/V of layer l and the K/V of the same decoder with bfloat16 storage of
    activations and cache (the floor of any two-byte pipeline); d[l] = relative L2 between two realisations of that
    pipeline that differ only in summation precision (how far two correct implementations drift apart)."""
    rows = []
    with open(os.path.join(GOLDEN, "bf16_depth_curve_8b.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([float(v) for v in line.split()])
    a = np.array(rows)
    return np.maximum(a[:, 1], a[:, 2]), np.maximum(a[:, 3], a[:, 4])


def _extend(curve, l):
    """curve[l], continued beyond its last entry with the square-root growth the whole curve shows."""
    last = len(curve) - 1
    return float(curve[l]) if l <= last else float(curve[last] * np.sqrt((l + 1.0) / (last + 1.0)))


STATED_REL_L2 = 1e-2     # the stated relative-L2 tolerance for bf16 K/V and next-token logits
STATED_MAX_ABS = 2e-2


def exact_bound(l, floor=None):
    """Allowed relative L2 between a bf16 pipeline's K/V at layer l (or logits after l layers) and the exact
    oracle: 1.5 x the oracle-only floor of that depth, and never looser than the stated tolerance where the
    floor leaves room for it (layers 0 and 1 of most shapes).  `floor` is the distance the oracle itself shows
    between its exact and its bf16-storage evaluation: by default the golden curve's value for layer l; a test
    that runs both evaluations on its own inputs passes what it measured (the floor moves a little with the
    shape and the context length)."""
    if floor is None:
        floor = _extend(depth_curve()[0], l)
    b = 1.5 * floor
    return STATED_REL_L2 if floor * 1.15 <= STATED_REL_L2 <= b else b


def oracle_floor(k_bf16, v_bf16, k_exact, v_exact, l):
    """Relative L2 of the oracle's bf16-storage K/V of layer l against its exact K/V over the rows both cover."""
    n = min(k_bf16.shape[1], k_exact.shape[1])
    return max(error_stats(k_bf16[l, :n], k_exact[l, :n])["rel_l2"], error_stats(v_bf16[l, :n], v_exact[l, :n])["rel_l2"])


def storage_bound(l):
    """Allowed relative L2 against the oracle evaluated with the same bfloat16 storage points: 2 x the drift between
    two correct realisations at that depth, plus 1e-3 for fp32 norm statistics, fp32 sin/cos and fp32 softmax."""
    return 1e-3 + 2.0 * _extend(depth_curve()[1], l)


class LockstepOracle:
    """Advances oracle forwards layer by layer while a model's weights are generated for upload, so that every
    layer's weights are drawn once and never all held on the host.  Pass `layers` to the binding's Model; after
    the model is built, `result(name)` returns (K, V, logits) of each registered evaluation."""

    def __init__(self, shape, seed, ids):
        self.shape, self.seed, self.ids = shape, seed, np.asarray(ids)
        self.head = synth.head_weights(shape, seed)
        self.runs = {}

    def add(self, name, n_tokens=None, act_bf16=False, mm_dtype=np.float32, want_logits=True, ids=None):
        """Registers a forward over the first n_tokens of the scenario's ids (or over `ids`, another request of
        the same model), positions 0 .. len - 1."""
        ids = self.ids[:n_tokens] if ids is None else np.asarray(ids)
        x = np.asarray(self.head["embed"], dtype=np.float64)[ids]
        self.runs[name] = dict(x=x, n=len(ids), act_bf16=act_bf16, mm=mm_dtype, k=[], v=[], logits=want_logits)
        return self

    def layers(self, l):
        w = synth.layer_weights(self.shape, self.seed, l)
        for r in self.runs.values():
            last = l == self.shape.n_layers - 1 and not r["logits"]
            r["x"], k, v = O.layer_forward(self.shape, w, r["x"], np.arange(r["n"]), mm_dtype=r["mm"],
                                           skip_after_kv=last, act_bf16=r["act_bf16"])
            r["k"].append(k)
            r["v"].append(v)
        return w

    def result(self, name):
        r = self.runs[name]
        assert len(r["k"]) == self.shape.n_layers, "build the model first: the oracle advances with the weight upload"
        logits = None
        if r["logits"]:
            logits = O._mm(O.rmsnorm(r["x"][-1:], self.head["final_norm"], self.shape.rms_eps), self.head["lm_head"],
                           r["mm"])[0]
        return np.stack(r["k"]), np.stack(r["v"]), logits


def _layer_source(shape, seed):
    cache = {}

    def layers(l):
        if l not in cache:
            cache.clear()
            cache[l] = synth.layer_weights(shape, seed, l)
        return cache[l]
    return layers


def oracle_reference(shape, seed, ids, mm_dtype=np.float64):
    """The exact definition: full forward over all ids."""
    head = synth.head_weights(shape, seed)
    K, V, logits = O.forward_full(shape, head, _layer_source(shape, seed), ids, mm_dtype=mm_dtype)
    return K, V, logits


def oracle_reference_bf16_storage(shape, seed, ids, k, mm_dtype=np.float64):
    """The same scenario evaluated by the oracle at the pipeline's storage precision: the prefix by a
    full forward with bf16 storage points, the suffix and the resumed token by incremental steps on a cache
    holding bf16 values (the cache element type is two bytes)."""
    head = synth.head_weights(shape, seed)
    layers = _layer_source(shape, seed)
    n = len(ids) - 1
    Kp, Vp, _ = O.forward_full(shape, head, layers, ids[:k], mm_dtype=mm_dtype, want_logits=False, act_bf16=True)
    L, _, hkv, d = Kp.shape
    Kc = np.zeros((L, n + 1, hkv, d)); Vc = np.zeros((L, n + 1, hkv, d))
    Kc[:, :k], Vc[:, :k] = Kp, Vp
    # held as fp64 once: the incremental step would otherwise convert every matrix on every call
    all_layers = [{k: np.asarray(v, dtype=np.float64) for k, v in synth.layer_weights(shape, seed, l).items()}
                  for l in range(shape.n_layers)]
    logits = None
    for pos in range(k, n + 1):
        kn, vn, logits = O.decode_step(shape, head, lambda l: all_layers[l], ids[pos], pos, Kc, Vc)
        Kc[:, pos] = O.from_bf16_bits(O.to_bf16_bits(kn))
        Vc[:, pos] = O.from_bf16_bits(O.to_bf16_bits(vn))
    return Kc, Vc, logits


def elementwise_ok(got, ref, rel_bound):
    """Element-wise form of a relative-L2 bound for values stored in bfloat16: the final rounding of a stored value
    moves it by at most half an ulp (<= 2^-8 |ref|), and what the bound allows as root-mean-square error may reach
    6 sigma on single elements of a tensor of millions.  (A literal max-abs of 2e-2 cannot hold on the wide shapes:
    K/V entries beyond |4| have a half-ulp of 0.0156 before any other error is counted.)"""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    return bool(np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 6.0 * rel_bound * rms))


def error_stats(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    return {
        "max_abs": float(err.max()),
        "rel_l2": float(np.sqrt(np.sum((got - ref) ** 2) / max(np.sum(ref ** 2), 1e-300))),
        "n_above_2e-2": int(np.sum(err > 2e-2)),
        "scaled_ok": bool(np.all(err <= 2e-2 * np.maximum(1.0, np.abs(ref) / 4.0))),
        "max_ref": float(np.abs(ref).max()),
    }


def run_gpu_scenario(kv, shape, seed, ids, k, n, num_blocks=64, cache_layout="layer_major", wire_layout=0, model=None):
    """Runs the whole path on the GPU through the C ABI.  Returns a dict of host arrays."""
    import torch
    bs = shape.block_size
    if model is None:
        head = synth.head_weights(shape, seed)
        model = kv.Model(shape, head, lambda l: synth.layer_weights(shape, seed, l))
    perm_src = synth.block_permutation(seed + 1, num_blocks)
    perm_tgt = synth.block_permutation(seed + 2, num_blocks)
    nb_total = -(-n // bs)
    nb_prefix = k // bs
    src = kv.PagedCache(shape, num_blocks, layout=cache_layout, fill=0)
    tgt = kv.PagedCache(shape, num_blocks, layout=cache_layout, fill=0)
    src_table = perm_src[:nb_total]
    # source: prefill the prefix, then produce the suffix token by token
    ws = kv.kv_prefill_prefix(model, src, ids[:k], src_table[:nb_prefix])
    kv.kv_check_device_status(ws)
    logits = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    for pos in range(k, n):
        kv.kv_decode_step(model, src, int(ids[pos]), pos, src_table[: pos // bs + 1], logits)
    # target: reconstruct the prefix locally
    tgt_prefix = perm_tgt[:nb_prefix]
    prefill_logits = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    ws = kv.kv_prefill_prefix(model, tgt, ids[:k], tgt_prefix, logits_out=prefill_logits)
    kv.kv_check_device_status(ws)
    # pack at the source, unpack + assemble at the target
    n_suffix = nb_total - nb_prefix
    wire = torch.zeros(n_suffix * shape.n_layers * 2 * (src.page_bytes // 2), dtype=torch.int16, device="cuda")
    kv.kv_pack_blocks(src, src_table[nb_prefix:], wire, wire_layout=wire_layout)
    dst_ids = perm_tgt[nb_prefix:nb_total]
    merged = kv.kv_unpack_assemble(tgt, wire, np.arange(nb_prefix, nb_total), dst_ids, tgt_prefix, n,
                                   epoch=7, expected_epoch=7, wire_layout=wire_layout)
    torch.cuda.synchronize()
    tgt_after_unpack = tgt.as_logical_numpy()     # before the resumed token is appended
    table = list(merged)
    if n % bs == 0:
        table.append(int(perm_tgt[nb_total]))      # the resumed token opens a new block
    kv.kv_decode_step(model, tgt, int(ids[n]), n, table, logits)
    torch.cuda.synchronize()
    tgt_img = tgt.as_logical_numpy()
    src_img = src.as_logical_numpy()
    Kg, Vg = O.read_kv(tgt_img, table, n + 1)
    return {
        "K": Kg, "V": Vg, "logits": logits.cpu().numpy(), "prefill_logits": prefill_logits.cpu().numpy(),
        "merged": merged, "expected_merged": np.concatenate([tgt_prefix, dst_ids]),
        "wire": wire.cpu().numpy().view(np.uint16), "src_img": src_img, "tgt_img": tgt_img, "tgt_after_unpack": tgt_after_unpack,
        "src_suffix_ids": src_table[nb_prefix:], "dst_ids": dst_ids, "table": table,
    }
