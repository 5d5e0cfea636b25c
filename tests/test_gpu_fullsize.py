"""Parity at the benchmark's full sizes and launch configuration.

The oracle cannot run 64 layers of the 32B shape in test time, so at that size the checks are (a) properties that
hold at any size and (b) sampled outputs the oracle computes one by one:
  * causality: the K/V pages a 4,096-token prefill leaves for its first 2,048 positions are byte-identical to
    those of a 2,048-token prefill (every kernel's per-row arithmetic is independent of later rows);
  * consistency of the two CUDA paths: decode_step(t[n]) on the assembled cache agrees with the last-row logits
    of a prefill over t[0..n];
  * pack/unpack: sampled pages of the 128 MiB wire and of the destination cache equal the host-generated
    counter pattern of the source pages, the merged table is the oracle's, untouched blocks stay zero.
The 8B shape (36 layers, 1,024 + 256 tokens) is checked at FULL depth against the oracle, and the 32B shape at the
benchmark's prefix and suffix lengths at reduced depth (two layers).
"""
import numpy as np
import pytest

import synth
from oracle import kv_oracle as O
from tests.scenario import (LockstepOracle, elementwise_ok, error_stats, exact_bound, oracle_floor,
                            run_gpu_scenario, storage_bound)

pytestmark = pytest.mark.gpu



@pytest.fixture(scope="module")
def kv():
    import paper_2608_16477_b200 as kv
    kv.load()
    return kv


def _device_model(kv, shape, seed):
    import torch
    gen = torch.Generator(device="cuda").manual_seed(seed)

    def mat(r, c):
        return torch.empty(r, c, dtype=torch.bfloat16, device="cuda").normal_(0.0, shape.init_std, generator=gen)
    ones = lambda: torch.ones(shape.hidden, dtype=torch.bfloat16, device="cuda")
    layer = lambda l: {"attn_norm": ones(), "ffn_norm": ones(), "w_qkv": mat(shape.qkv_dim, shape.hidden),
                       "w_o": mat(shape.hidden, shape.q_dim), "w_gate_up": mat(2 * shape.ffn, shape.hidden),
                       "w_down": mat(shape.hidden, shape.ffn)}
    head = {"embed": mat(shape.vocab, shape.hidden), "lm_head": mat(shape.vocab, shape.hidden), "final_norm": ones()}
    return kv.Model(shape, head, layer)


def test_32b_full_depth_properties(kv):
    import torch
    s = synth.SHAPES["32b"]
    prefix, suffix, pool = 4096, 512, 4096          # the benchmark's configuration
    n = prefix + suffix
    bs = s.block_size
    model = _device_model(kv, s, 7)
    ids = synth.token_ids(s, 7, n + 1)
    perm = synth.block_permutation(8, pool)
    cache = kv.PagedCache(s, pool, fill=0)
    nb = prefix // bs
    # (a) causality at full size: prefill(4096) vs prefill(2048) into disjoint blocks
    t_full, t_half = perm[:nb], perm[nb:nb + nb // 2]
    ws = kv.kv_prefill_prefix(model, cache, ids[:prefix], t_full)
    kv.kv_check_device_status(ws)
    ws = kv.kv_prefill_prefix(model, cache, ids[:prefix // 2], t_half)
    kv.kv_check_device_status(ws)
    a = cache.pages(t_full[: nb // 2])
    b = cache.pages(t_half)
    assert torch.equal(a, b), "K/V of the first half depend on later tokens"
    assert bool(a.any())
    # (b) decode step on the cache vs prefill-with-logits over one more token
    lg_dec = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    table = list(perm[:nb]) + [int(perm[nb + nb // 2])]
    kv.kv_decode_step(model, cache, int(ids[prefix]), prefix, table, lg_dec)
    lg_pre = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    t2 = perm[2 * nb: 3 * nb + 1]
    kv.kv_prefill_prefix(model, cache, ids[:prefix + 1], t2, logits_out=lg_pre)
    torch.cuda.synchronize()
    st = error_stats(lg_dec.cpu().numpy(), lg_pre.cpu().numpy())
    print("decode vs prefill logits at depth 64:", st)
    # the decode path keeps fp32 activations, the prefill path stores them in bf16: the two differ by at most the
    # bf16 storage noise accumulated over 64 layers (the oracle-only floor of that depth; measured 4.6 %)
    assert st["rel_l2"] <= exact_bound(s.n_layers), (st, exact_bound(s.n_layers))
    # the appended K/V row of the decode step equals the prefill's row for that position up to bf16 rounding
    # slot 0 of the block opened for position 4096 (int16 bit patterns viewed as bf16 values)
    ka = cache.pages([table[-1]])[0, :, :, : s.n_kv_heads * s.head_dim].contiguous().view(torch.bfloat16).float()
    kb = cache.pages([int(t2[-1])])[0, :, :, : s.n_kv_heads * s.head_dim].contiguous().view(torch.bfloat16).float()
    rel = (torch.linalg.norm(ka - kb) / torch.linalg.norm(kb)).item()
    assert rel <= exact_bound(s.n_layers), rel


def test_32b_full_depth_single_layers_against_oracle(kv):
    """Single layers of the 64-layer 32B-shaped model at the benchmark's prefix length, each against the oracle on that
    layer's TRUE input.

    The oracle cannot run 64 layers of this shape in test time, but it can run ONE layer of it.  A K/V-only prefill of
    the first l + 1 layers leaves the input x_l of layer l in the workspace's residual stream and that layer's K/V in
    the cache; the same prefill with logits leaves the layer's output x_{l+1}.  The oracle evaluates the layer on the
    GPU's own x_l (all 4,096 rows), so nothing accumulates and the bounds are those of a first layer:
      * K/V of layers 1, 15, 31, 47 and 63 within exact_bound(0) of the oracle (3.5e-3; the floor of two-byte storage is 2.35e-3);
      * the update x_{l+1} - x_l of the LAST layer (attention, O projection, SwiGLU FFN at K = 8,192 and 25,600 in the
        benchmark's instantiations) within 1.5 x the distance the oracle's own bf16-storage evaluation has from its exact
        one, and close to that bf16-storage evaluation."""
    import torch
    s = synth.SHAPES["32b"]
    s = synth.ModelShape(**{**s.__dict__, "vocab": 4096})
    prefix = 4096
    bs = s.block_size
    gen = torch.Generator(device="cuda").manual_seed(11)

    def mat(r, c):
        return torch.empty(r, c, dtype=torch.bfloat16, device="cuda").normal_(0.0, s.init_std, generator=gen)
    ones = lambda: torch.ones(s.hidden, dtype=torch.bfloat16, device="cuda")
    W = [{"attn_norm": ones(), "ffn_norm": ones(), "w_qkv": mat(s.qkv_dim, s.hidden), "w_o": mat(s.hidden, s.q_dim),
          "w_gate_up": mat(2 * s.ffn, s.hidden), "w_down": mat(s.hidden, s.ffn)} for _ in range(s.n_layers)]
    head = {"embed": mat(s.vocab, s.hidden), "lm_head": mat(s.vocab, s.hidden), "final_norm": ones()}
    ids = synth.token_ids(s, 11, prefix)
    table = synth.block_permutation(12, 512)[: prefix // bs]
    pos = np.arange(prefix)
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")

    def residual(model, ws):
        off, nbytes = kv.kv_workspace_residual(model, kv.KV_OP_PREFILL, prefix)
        return ws[off:off + nbytes].view(torch.float32).view(prefix, s.hidden).cpu().numpy().astype(np.float64)

    for l, whole_layer in ((1, False), (15, False), (31, False), (47, False), (63, True)):
        sub = s.with_layers(l + 1)
        model = kv.Model(sub, head, lambda i: W[i])             # shares the device tensors, no copies
        cache = kv.PagedCache(sub, 512, fill=0)
        ws = kv.kv_prefill_prefix(model, cache, ids, table)      # K/V only: the last layer stops after its K/V
        kv.kv_check_device_status(ws)
        x_in = residual(model, ws)
        img = cache.data[l].cpu().numpy().view(np.uint16).reshape(1, 2, 512, bs, s.n_kv_heads, s.head_dim)
        Kg, Vg = O.read_kv(img, table, prefix)
        w_host = {k: v.float().cpu().numpy() for k, v in W[l].items()}
        _, Kref, Vref = O.layer_forward(s, w_host, x_in, pos, mm_dtype=np.float32, skip_after_kv=True)
        for nm, got, ref in (("K", Kg[0], Kref), ("V", Vg[0], Vref)):
            st = error_stats(got, ref)
            print(f"32b layer {l} {nm} on its true input:", st)
            assert st["rel_l2"] <= exact_bound(0) and elementwise_ok(got, ref, exact_bound(0)), (l, nm, st)
        if not whole_layer:
            continue
        ws = kv.kv_prefill_prefix(model, cache, ids, table, logits_out=logits)     # now the last layer runs to its end
        kv.kv_check_device_status(ws)
        x_out = residual(model, ws)
        xe, _, _ = O.layer_forward(s, w_host, x_in, pos, mm_dtype=np.float32)
        xb, _, _ = O.layer_forward(s, w_host, x_in, pos, mm_dtype=np.float32, act_bf16=True)
        u_ref = xe - x_in
        norm = float(np.sqrt(np.sum(u_ref ** 2)))
        floor = float(np.sqrt(np.sum((xb - xe) ** 2))) / norm
        vs_exact = float(np.sqrt(np.sum((x_out - xe) ** 2))) / norm
        vs_storage = float(np.sqrt(np.sum((x_out - xb) ** 2))) / norm
        print(f"32b layer {l} update x_out - x_in: oracle floor {floor:.4e}, GPU vs exact {vs_exact:.4e}, "
              f"GPU vs bf16-storage oracle {vs_storage:.4e}, |update| / |x| {norm / np.sqrt(np.sum(x_in ** 2)):.3e}")
        assert vs_exact <= 1.5 * floor, (vs_exact, floor)
        assert vs_storage <= floor, (vs_storage, floor)


def test_32b_full_size_pack_unpack_sampled(kv):
    import torch
    s = synth.SHAPES["32b"]
    pool, n_blocks = 4096, 32                      # 16 GiB pools, 128 MiB payload: the benchmark's launch
    src = kv.PagedCache(s, pool)
    kv.kv_fill_pattern(src.data, src.data.numel() * 2, seed=1234)
    dst = kv.PagedCache(s, pool, fill=0)
    ids_src = synth.block_permutation(21, pool)[256:256 + n_blocks]
    ids_dst = synth.block_permutation(22, pool)[256:256 + n_blocks]
    prefix = synth.block_permutation(22, pool)[:256]
    page = src.page_bytes
    wire = torch.empty(n_blocks * s.n_layers * 2 * page, dtype=torch.uint8, device="cuda")
    kv.kv_pack_blocks(src, ids_src, wire)
    n_tokens = (256 + n_blocks) * s.block_size - 5
    merged = kv.kv_unpack_assemble(dst, wire, np.arange(256, 256 + n_blocks), ids_dst, prefix, n_tokens)
    torch.cuda.synchronize()
    st, want_merged = O.OK, np.concatenate([prefix, ids_dst])
    assert O.check_assemble(pool, s.block_size, np.arange(256, 256 + n_blocks), ids_dst, prefix, n_tokens, 0, 0) == O.OK
    assert np.array_equal(merged, want_merged)
    rng = np.random.default_rng(3)
    for _ in range(64):
        i = int(rng.integers(0, n_blocks)); l = int(rng.integers(0, s.n_layers)); kvi = int(rng.integers(0, 2))
        src_off = ((l * 2 + kvi) * pool + int(ids_src[i])) * page
        want = synth.pattern_bytes(1234, src_off, page)          # what the oracle's pack would copy
        w_off = ((i * s.n_layers + l) * 2 + kvi) * page
        assert np.array_equal(wire[w_off:w_off + page].cpu().numpy(), want)
        assert np.array_equal(dst.data[l, kvi, int(ids_dst[i])].cpu().numpy().view(np.uint8), want)
    # untouched destination blocks: a sample of blocks outside ids_dst is still zero
    others = np.setdiff1d(np.arange(pool), ids_dst)[:: 97]
    assert not dst.data[:, :, torch.from_numpy(others).cuda()].any()
    # whole-wire checksum against the destination pages (every byte, on the device)
    got = dst.pages(ids_dst).contiguous().view(torch.uint8).reshape(-1)
    assert torch.equal(got, wire)


def _per_layer(got_k, got_v, ref_k, ref_v, lo=0, hi=None):
    rows = []
    for l in range(got_k.shape[0]):
        rows.append((error_stats(got_k[l, lo:hi], ref_k[l, lo:hi])["rel_l2"], error_stats(got_v[l, lo:hi], ref_v[l, lo:hi])["rel_l2"]))
    return rows


def test_8b_full_depth_against_oracle(kv):
    """The 8B-shaped configuration as written: 36 layers, prefix 1,024 + suffix 256, single request, at FULL depth.

    The oracle advances in lockstep with the weight upload (exact definition over all 1,281 tokens; the same
    function with bfloat16 storage points over the prefix).  Three claims per layer:
      * against the exact oracle the K/V stay within 1.5 x the floor that the oracle alone shows for two-byte
        storage at that depth (tests/golden/bf16_depth_curve_8b.txt; the stated 1e-2 wherever the floor allows it);
      * against the storage-precision oracle the prefix K/V stay within the drift of two correct realisations;
      * pack / unpack / assemble are bit-exact, as everywhere."""
    s = synth.SHAPES["8b"]
    s = synth.ModelShape(**{**s.__dict__, "vocab": 8192})
    k, n = 1024, 1024 + 256
    ids = synth.token_ids(s, 0, n + 1)
    lock = LockstepOracle(s, 0, ids).add("exact", n + 1).add("bf16", k, act_bf16=True, want_logits=False)
    model = kv.Model(s, lock.head, lock.layers)
    res = run_gpu_scenario(kv, s, 0, ids, k, n, num_blocks=256, model=model)
    assert np.array_equal(res["merged"], res["expected_merged"])
    want_wire = O.pack_blocks(res["src_img"], res["src_suffix_ids"])
    assert np.array_equal(res["wire"], want_wire.reshape(-1))
    for s_id, d_id in zip(res["src_suffix_ids"], res["dst_ids"]):
        assert np.array_equal(res["tgt_after_unpack"][:, :, d_id], res["src_img"][:, :, s_id])
    Kref, Vref, logits_ref = lock.result("exact")
    Kb, Vb, _ = lock.result("bf16")
    exact = _per_layer(res["K"], res["V"], Kref, Vref)
    prefix = _per_layer(res["K"], res["V"], Kb, Vb, 0, k)
    lg = error_stats(res["logits"], logits_ref)
    print("8b full depth, per-layer (K, V) rel_l2 vs exact:", [(round(a, 5), round(b, 5)) for a, b in exact])
    print("8b full depth, prefix per-layer (K, V) rel_l2 vs bf16-storage oracle:", [(round(a, 5), round(b, 5)) for a, b in prefix])
    print("8b full depth logits vs exact:", lg, "bound", exact_bound(s.n_layers))
    floors = [oracle_floor(Kb, Vb, Kref, Vref, l) for l in range(s.n_layers)]
    print("8b full depth, oracle floor (bf16-storage vs exact) on these inputs:", [round(f, 5) for f in floors])
    for l in range(s.n_layers):
        # both the golden curve (256 tokens) and the floor measured on these 1,024 prefix tokens must hold
        assert max(exact[l]) <= exact_bound(l, floors[l]), (l, exact[l], floors[l])
        assert max(exact[l]) <= exact_bound(l), (l, exact[l], exact_bound(l))
        assert max(prefix[l]) <= storage_bound(l), (l, prefix[l], storage_bound(l))
    assert lg["rel_l2"] <= exact_bound(s.n_layers), lg


def test_32b_bench_launch_configuration_against_oracle(kv):
    """The whole scenario at the benchmark's own launch configuration (32B shape, prefix 4,096 + suffix 512, pools of
    4,096 blocks, fragmented ids) at reduced depth against the oracle.  The projections must run the instantiations the
    benchmark runs: CTA pairs with 256-wide tiles for QKV and gate/up, 224-wide for the O and down projections
    (K = 8,192 and 25,600)."""
    s = synth.SHAPES["32b"].with_layers(2)
    s = synth.ModelShape(**{**s.__dict__, "vocab": 4096})
    prefix, suffix, pool = 4096, 512, 4096
    n = prefix + suffix
    assert kv.kv_gemm_plan(prefix, s.qkv_dim, 3, head_dim=s.head_dim) == (True, 256)
    assert kv.kv_gemm_plan(prefix, s.hidden, 1) == (True, 224)
    assert kv.kv_gemm_plan(prefix, s.ffn, 2) == (True, 256)
    ids = synth.token_ids(s, 0, n + 1)
    lock = LockstepOracle(s, 0, ids).add("exact", n + 1).add("bf16", prefix, act_bf16=True, want_logits=False)
    model = kv.Model(s, lock.head, lock.layers)
    res = run_gpu_scenario(kv, s, 0, ids, prefix, n, num_blocks=pool, model=model)
    assert np.array_equal(res["merged"], res["expected_merged"])
    want_wire = O.pack_blocks(res["src_img"], res["src_suffix_ids"])
    assert np.array_equal(res["wire"], want_wire.reshape(-1))
    for s_id, d_id in zip(res["src_suffix_ids"], res["dst_ids"]):
        assert np.array_equal(res["tgt_after_unpack"][:, :, d_id], res["src_img"][:, :, s_id])
    Kref, Vref, logits_ref = lock.result("exact")
    Kb, Vb, _ = lock.result("bf16")
    report = {}
    for l in range(2):
        # the floor of two-byte storage for THIS shape and context length, from the two oracle evaluations
        floor = oracle_floor(Kb, Vb, Kref, Vref, l)
        report[f"oracle_floor{l}"] = floor
        for nm, got, ref, refb in (("K", res["K"][l], Kref[l], Kb[l]), ("V", res["V"][l], Vref[l], Vb[l])):
            st = error_stats(got, ref)
            report[f"exact_{nm}{l}"] = st
            bound = exact_bound(l, floor)
            assert st["rel_l2"] <= bound and elementwise_ok(got, ref, bound), (l, nm, st, floor, bound)
            sb = error_stats(got[:prefix], refb)
            report[f"storage_{nm}{l}"] = sb
            assert sb["rel_l2"] <= storage_bound(l), (l, nm, sb)
            rms = float(np.sqrt(np.mean(np.asarray(refb, dtype=np.float64) ** 2)))
            assert np.all(np.abs(got[:prefix] - refb) <= 8 * storage_bound(l) * rms + 2.0 ** -7 * np.abs(refb)), (l, nm, sb)
    report["logits"] = error_stats(res["logits"], logits_ref)
    print("32b x 2 layers at 4096 + 512:", report)
    assert report["logits"]["rel_l2"] <= exact_bound(2), report["logits"]


def test_pack_unpack_stress_16_requests_full_size(kv):
    """The 16-request stress workload at full size: 4,639 blocks (18.1 GiB) gathered from a source pool of up to
    32,768 blocks into per-request wire buffers and scattered into a second cache, in the batched launch form.
    Sampled pages are checked against the host-generated counter pattern (what the oracle's pack would copy)."""
    import torch
    from bench import stress_geometry
    s = synth.SHAPES["32b"]
    counts, total, src_blocks, dst_blocks, block_bytes = stress_geometry(kv, torch, s)
    assert total == 4639 and total * block_bytes == 4639 * 4 * 1024 * 1024
    page = synth.kv_page_bytes(s)
    src = kv.PagedCache(s, src_blocks)
    dst = kv.PagedCache(s, dst_blocks, fill=0)
    kv.kv_fill_pattern(src.data, src.data.numel() * 2, seed=77)
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    src_ids = synth.block_permutation(1, src_blocks)[:total]
    dst_ids = synth.block_permutation(2, dst_blocks)[:total]
    wires = [torch.empty(c * block_bytes, dtype=torch.uint8, device="cuda") for c in counts]
    kv.kv_pack_blocks_batched(src, offs, src_ids, wires)
    kv.kv_unpack_blocks_batched(dst, offs, dst_ids, wires)
    kv.kv_check_copy_status()
    rng = np.random.default_rng(9)
    for _ in range(96):
        r = int(rng.integers(0, len(counts))); i = int(rng.integers(0, counts[r]))
        l = int(rng.integers(0, s.n_layers)); kvi = int(rng.integers(0, 2))
        b_src, b_dst = int(src_ids[offs[r] + i]), int(dst_ids[offs[r] + i])
        want = synth.pattern_bytes(77, ((l * 2 + kvi) * src_blocks + b_src) * page, page)
        w_off = ((i * s.n_layers + l) * 2 + kvi) * page
        assert np.array_equal(wires[r][w_off:w_off + page].cpu().numpy(), want)
        assert np.array_equal(dst.data[l, kvi, b_dst].cpu().numpy().view(np.uint8), want)
    unused = np.setdiff1d(np.arange(dst_blocks), dst_ids)
    assert not dst.data[:, :, torch.from_numpy(unused).cuda()].any()
    print("stress geometry:", dict(src_blocks=src_blocks, dst_blocks=dst_blocks, blocks=total))
