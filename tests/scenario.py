"""Shared driver of the end-to-end parity scenario (test helper; imports both the oracle and the binding).

tokens t[0..n] (n+1 ids, teacher-forced): the source cache is built by prefill(t[0:k]) followed by decode
steps for t[k..n-1]; the target cache by prefill(t[0:k]) into its own fresh blocks; the suffix blocks are
packed at the source, unpacked/assembled at the target, and the target resumes with decode_step(t[n], pos=n).
Reference values: the oracle's full forward over t[0..n].
"""
import numpy as np

import synth
from oracle import kv_oracle as O


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
    all_layers = [synth.layer_weights(shape, seed, l) for l in range(shape.n_layers)]
    logits = None
    for pos in range(k, n + 1):
        kn, vn, logits = O.decode_step(shape, head, lambda l: all_layers[l], ids[pos], pos, Kc, Vc)
        Kc[:, pos] = O.from_bf16_bits(O.to_bf16_bits(kn))
        Vc[:, pos] = O.from_bf16_bits(O.to_bf16_bits(vn))
    return Kc, Vc, logits


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


def run_gpu_scenario(kv, shape, seed, ids, k, n, num_blocks=64, cache_layout="layer_major", wire_layout=0):
    """Runs the whole path on the GPU through the C ABI.  Returns a dict of host arrays."""
    import torch
    bs = shape.block_size
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
