"""The variants of the path beyond the single-shot migration, each against the CPU oracle:

  * continued (chunked) prefill, `pos0 > 0` (Section 4.5: the migration prefill split into chunks that interleave
    with resident decoding; 256-token chunks in the handover-inference contention experiment, Section 6.3);
  * "without suffix migration" (Section 6.4 ablation): the target recomputes the suffix as a continued prefill
    from position k instead of receiving its blocks;
  * several prefix reconstructions in one call (Section 4.5 / 6.3: concurrent handovers sharing the target GPU);
  * Full-Copy (Section 2.2; Section 6.4 "without prefix recomputation"): every block of the request travels
    through pack and unpack, the target prefills nothing.
"""
import numpy as np
import pytest

import synth
from oracle import kv_oracle as O
from tests.scenario import (STATED_MAX_ABS, STATED_REL_L2, LockstepOracle, elementwise_ok, error_stats, exact_bound,
                            oracle_floor)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kv():
    import paper_2608_16477_b200 as kv
    kv.load()
    return kv


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _kv_of(cache, table, n):
    return O.read_kv(cache.as_logical_numpy(), table, n)


def _check_kv(shape, got_k, got_v, ref_k, ref_v, literal, what, floors=None):
    for l in range(shape.n_layers):
        bound = exact_bound(l, None if floors is None else floors[l])
        for nm, got, ref in (("K", got_k[l], ref_k[l]), ("V", got_v[l], ref_v[l])):
            st = error_stats(got, ref)
            assert st["rel_l2"] <= bound, (what, l, nm, st, bound)
            assert (st["max_abs"] <= STATED_MAX_ABS) if literal else elementwise_ok(got, ref, bound), (what, l, nm, st)


def _tiny_model(kv, name, seed):
    s = synth.SHAPES[name]
    head = synth.head_weights(s, seed)
    lw = [synth.layer_weights(s, seed, l) for l in range(s.n_layers)]
    return s, head, lw, kv.Model(s, head, lambda l: lw[l])


# ------------------------------------------------------------------ continued prefill against the oracle
@pytest.mark.parametrize("name", ["tiny", "tiny-sharp"])
@pytest.mark.parametrize("chunks", [(64, 96), (48, 16, 80, 16), (160,)])
def test_chunked_prefill_against_oracle_tiny(kv, torch, name, chunks):
    s, head, lw, model = _tiny_model(kv, name, 3)
    n = sum(chunks)
    ids = synth.token_ids(s, 3, n)
    Kref, Vref, lref = O.forward_full(s, head, lambda l: lw[l], ids)
    table = synth.block_permutation(4, 64)[: n // 16]
    cache = kv.PagedCache(s, 64, fill=0)
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    p0 = 0
    for i, c in enumerate(chunks):
        last = i == len(chunks) - 1
        ws = kv.kv_prefill_prefix(model, cache, ids[p0:p0 + c], table[: (p0 + c) // 16], pos0=p0,
                                  logits_out=logits if last else None)
        kv.kv_check_device_status(ws)
        p0 += c
    Kg, Vg = _kv_of(cache, table, n)
    _check_kv(s, Kg, Vg, Kref, Vref, name == "tiny", ("chunked", chunks))
    st = error_stats(logits.cpu().numpy(), lref)
    assert st["rel_l2"] <= STATED_REL_L2, st
    # pages outside the table stay untouched
    img = cache.as_logical_numpy()
    assert not img[:, :, np.setdiff1d(np.arange(64), table)].any()


@pytest.mark.parametrize("name", ["tiny", "tiny-sharp"])
def test_chunked_prefill_interleaved_with_resident_decode(kv, torch, name):
    """Section 4.5's schedule on one stream: a migrating request's prefix is rebuilt in chunks while a resident request
    on the same model and the same block pool decodes one token after every chunk.  Both are checked against the
    oracle: the resident request's logits at every step, the migrating request's K/V and first resumed token."""
    s, head, lw, model = _tiny_model(kv, name, 7)
    chunks = (48, 32, 16, 64)
    n_mig, n_res = sum(chunks), 80
    mig_ids = synth.token_ids(s, 8, n_mig + 1)
    res_ids = synth.token_ids(s, 9, n_res + len(chunks) + 1)
    Km, Vm, lm = O.forward_full(s, head, lambda l: lw[l], mig_ids)
    perm = synth.block_permutation(10, 64)
    res_table, mig_table = perm[:8], perm[8:8 + n_mig // 16 + 1]
    cache = kv.PagedCache(s, 64, fill=0)
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    kv.kv_prefill_prefix(model, cache, res_ids[:n_res], res_table[: n_res // 16])
    p0 = 0
    for i, c in enumerate(chunks):
        ws = kv.kv_prefill_prefix(model, cache, mig_ids[p0:p0 + c], mig_table[: (p0 + c) // 16], pos0=p0)
        kv.kv_check_device_status(ws)
        p0 += c
        pos = n_res + i
        kv.kv_decode_step(model, cache, int(res_ids[pos]), pos, res_table[: pos // 16 + 1], logits)
        _, _, lref = O.forward_full(s, head, lambda l: lw[l], res_ids[: pos + 1])
        st = error_stats(logits.cpu().numpy(), lref)
        assert st["rel_l2"] <= STATED_REL_L2, ("resident", i, st)
    Kg, Vg = _kv_of(cache, mig_table, n_mig)
    _check_kv(s, Kg, Vg, Km[:, :n_mig], Vm[:, :n_mig], name == "tiny", "interleaved")
    kv.kv_decode_step(model, cache, int(mig_ids[n_mig]), n_mig, mig_table, logits)
    st = error_stats(logits.cpu().numpy(), lm)
    assert st["rel_l2"] <= STATED_REL_L2, ("migrated", st)
    # the two requests' pages are disjoint and nothing else was written
    img = cache.as_logical_numpy()
    used = np.concatenate([res_table[: (n_res + len(chunks)) // 16 + 1], mig_table])
    assert not img[:, :, np.setdiff1d(np.arange(64), used)].any()


@pytest.fixture(scope="module")
def wide(kv):
    """A 32B-shaped two-layer model and the oracle's exact forward over 1,000 tokens (shared by the wide cases)."""
    s = synth.SHAPES["32b"].with_layers(2)
    s = synth.ModelShape(**{**s.__dict__, "vocab": 2048})
    n = 1000
    ids = synth.token_ids(s, 5, n + 1)
    # the second and third evaluations serve the batched case: requests are ids[:300] and ids[100:612]
    lock = LockstepOracle(s, 5, ids).add("exact", n + 1).add("first", 300).add("second", ids=ids[100:612])
    lock.add("bf16", n, act_bf16=True, want_logits=False)      # the floor of two-byte storage on these inputs
    model = kv.Model(s, lock.head, lock.layers)
    exact, bf16 = lock.result("exact"), lock.result("bf16")
    floors = [oracle_floor(bf16[0], bf16[1], exact[0], exact[1], l) for l in range(s.n_layers)]
    return dict(shape=s, n=n, ids=ids, model=model, exact=exact, first=lock.result("first"),
                second=lock.result("second"), floors=floors)


def test_chunked_prefill_against_oracle_wide(kv, torch, wide):
    """256-token chunks with a ragged tail (232 tokens) on the 32B shape: the cached prefix is gathered from its pages
    for the tensor-core attention kernel."""
    s, n, ids, model = wide["shape"], wide["n"], wide["ids"], wide["model"]
    Kref, Vref, _ = wide["exact"]
    table = synth.block_permutation(6, 128)[: -(-n // 16)]
    cache = kv.PagedCache(s, 128, fill=0)
    for p0 in range(0, n, 256):
        chunk = ids[p0:min(p0 + 256, n)]
        ws = kv.kv_prefill_prefix(model, cache, chunk, table[: -(-(p0 + len(chunk)) // 16)], pos0=p0)
        kv.kv_check_device_status(ws)
    Kg, Vg = _kv_of(cache, table, n)
    _check_kv(s, Kg, Vg, Kref[:, :n], Vref[:, :n], False, "chunked-wide", wide["floors"])
    # resume on the chunk-built cache: the decode step's logits against the exact last row
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    kv.kv_decode_step(model, cache, int(ids[n]), n, table, logits)
    st = error_stats(logits.cpu().numpy(), wide["exact"][2])
    assert st["rel_l2"] <= exact_bound(s.n_layers), st


# ------------------------------------------------------------------ host arrays belong to the caller again on return
def test_host_arrays_may_be_overwritten_as_soon_as_a_call_returns(kv, torch):
    """Token ids and block tables handed over in page-locked memory, with the stream still busy when the call returns,
    are overwritten at once with other (valid) values: prefill, batched prefill and decode step must have taken their
    own copy.  The reference results come from the same calls with untouched arrays."""
    s, head, lw, model = _tiny_model(kv, "tiny", 11)
    n = 96
    ids = synth.token_ids(s, 11, n + 1)
    table = synth.block_permutation(12, 64)[: n // 16 + 1]
    other_ids = synth.token_ids(s, 13, n + 1)
    other_table = synth.block_permutation(14, 64)[: n // 16 + 1]
    busy = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")

    def pinned(a):
        t = torch.from_numpy(np.asarray(a, dtype=np.int32).copy()).pin_memory()
        return t, t.numpy()

    def run(overwrite):
        cache = kv.PagedCache(s, 64, fill=0)
        lg = torch.zeros(3, s.vocab, dtype=torch.float32, device="cuda")
        keep = []
        def hand_over(a, b):
            t, view = pinned(a)
            keep.append(t)
            return view, np.asarray(b, dtype=np.int32)
        def clobber(*pairs):
            if overwrite:
                for view, repl in pairs:
                    view[:] = repl
        def delay():                                   # a few milliseconds of work ahead of the call in the stream
            for _ in range(12):
                kv.kv_fill_pattern(busy, busy.numel(), seed=1)
        i1, t1 = hand_over(ids[:n], other_ids[:n]), hand_over(table[: n // 16], other_table[: n // 16])
        delay()
        kv.kv_prefill_prefix(model, cache, i1[0], t1[0], logits_out=lg[0])
        clobber(i1, t1)
        t2 = hand_over(table, other_table)
        delay()
        kv.kv_decode_step(model, cache, int(ids[n]), n, t2[0], lg[1])
        clobber(t2)
        # the batched form into other pages of the same cache
        free = np.setdiff1d(np.arange(64), table)[: n // 16]
        i3, t3 = hand_over(ids[:n], other_ids[:n]), hand_over(free, free[::-1].copy())
        delay()
        kv.kv_prefill_prefix_batched(model, cache, [i3[0]], [t3[0]], logits_out=lg[2:3])
        clobber(i3, t3)
        torch.cuda.synchronize()
        return cache.data.clone(), lg.clone()

    ref_cache, ref_lg = run(False)
    got_cache, got_lg = run(True)
    assert bool(ref_cache.any()) and torch.equal(got_cache, ref_cache)
    assert torch.equal(got_lg, ref_lg)


# ------------------------------------------------------------------ "without suffix migration"
@pytest.mark.parametrize("name", ["tiny", "tiny-sharp"])
def test_suffix_recomputed_at_target_tiny(kv, torch, name):
    """The target rebuilds the prefix, then recomputes the suffix [k, n) itself as a continued prefill (no blocks
    travel) and resumes at n: K/V of every position and the next-token logits against the oracle's full forward."""
    s, head, lw, model = _tiny_model(kv, name, 0)
    k, n = 128, 165
    ids = synth.token_ids(s, 0, n + 1)
    Kref, Vref, lref = O.forward_full(s, head, lambda l: lw[l], ids)
    table = synth.block_permutation(2, 64)[: -(-(n + 1) // 16)]
    cache = kv.PagedCache(s, 64, fill=0)
    kv.kv_prefill_prefix(model, cache, ids[:k], table[: k // 16])
    kv.kv_prefill_prefix(model, cache, ids[k:n], table[: -(-n // 16)], pos0=k)
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    kv.kv_decode_step(model, cache, int(ids[n]), n, table, logits)
    Kg, Vg = _kv_of(cache, table, n + 1)
    _check_kv(s, Kg, Vg, Kref, Vref, name == "tiny", "recomputed-suffix")
    st = error_stats(logits.cpu().numpy(), lref)
    assert st["rel_l2"] <= STATED_REL_L2 and st["max_abs"] <= (STATED_MAX_ABS if name == "tiny" else np.inf), st


def test_suffix_recomputed_at_target_wide(kv, torch, wide):
    s, n, ids, model = wide["shape"], wide["n"], wide["ids"], wide["model"]
    Kref, Vref, lref = wide["exact"]
    k = 768
    table = synth.block_permutation(7, 128)[: -(-(n + 1) // 16)]
    cache = kv.PagedCache(s, 128, fill=0)
    kv.kv_prefill_prefix(model, cache, ids[:k], table[: k // 16])
    ws = kv.kv_prefill_prefix(model, cache, ids[k:n], table[: -(-n // 16)], pos0=k)
    kv.kv_check_device_status(ws)
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    kv.kv_decode_step(model, cache, int(ids[n]), n, table, logits)
    Kg, Vg = _kv_of(cache, table, n + 1)
    _check_kv(s, Kg, Vg, Kref, Vref, False, "recomputed-suffix-wide", wide["floors"])
    st = error_stats(logits.cpu().numpy(), lref)
    assert st["rel_l2"] <= exact_bound(s.n_layers), st


# ------------------------------------------------------------------ batched prefill against the oracle
def test_batched_prefill_against_oracle_tiny(kv, torch):
    s, head, lw, model = _tiny_model(kv, "tiny-sharp", 9)
    lengths = (100, 37, 260)
    perm = synth.block_permutation(10, 256)
    ids, tables, used = [], [], 0
    for i, n in enumerate(lengths):
        ids.append(synth.token_ids(s, 20 + i, n))
        nb = -(-n // s.block_size)
        tables.append(perm[used:used + nb].copy())
        used += nb
    cache = kv.PagedCache(s, 256, fill=0)
    logits = torch.zeros(len(lengths), s.vocab, dtype=torch.float32, device="cuda")
    ws = kv.kv_prefill_prefix_batched(model, cache, ids, tables, logits_out=logits)
    kv.kv_check_device_status(ws)
    for i, n in enumerate(lengths):
        Kref, Vref, lref = O.forward_full(s, head, lambda l: lw[l], ids[i])
        Kg, Vg = _kv_of(cache, tables[i], n)
        _check_kv(s, Kg, Vg, Kref, Vref, False, ("batched", i))
        st = error_stats(logits[i].cpu().numpy(), lref)
        assert st["rel_l2"] <= STATED_REL_L2, (i, st)
    img = cache.as_logical_numpy()
    assert not img[:, :, perm[used:]].any()


def test_batched_prefill_against_oracle_wide(kv, torch, wide):
    """Two requests of the 32B shape (300 and 512 tokens, different token ids) in one call: all 812 rows share the
    projection launches, attention runs per request; each request against its own oracle forward."""
    s, ids, model = wide["shape"], wide["ids"], wide["model"]
    reqs = [ids[:300], ids[100:612]]
    perm = synth.block_permutation(11, 128)
    tables = [perm[:19].copy(), perm[19:19 + 32].copy()]
    cache = kv.PagedCache(s, 128, fill=0)
    logits = torch.zeros(2, s.vocab, dtype=torch.float32, device="cuda")
    ws = kv.kv_prefill_prefix_batched(model, cache, reqs, tables, logits_out=logits)
    kv.kv_check_device_status(ws)
    for i, key in enumerate(("first", "second")):
        Kref, Vref, lref = wide[key]
        Kg, Vg = _kv_of(cache, tables[i], len(reqs[i]))
        _check_kv(s, Kg, Vg, Kref, Vref, False, ("batched-wide", i), wide["floors"])
        st = error_stats(logits[i].cpu().numpy(), lref)
        assert st["rel_l2"] <= exact_bound(s.n_layers), (i, st)


# ------------------------------------------------------------------ Full-Copy
@pytest.mark.parametrize("name,n", [("tiny", 160), ("tiny-sharp", 149)])
@pytest.mark.parametrize("wire_layout", [0, 1])
def test_full_copy_rebuilds_cache_from_the_wire_alone(kv, torch, name, n, wire_layout):
    """Every block of the request goes through kv_pack_blocks; the target starts from an empty cache, prefills
    nothing (n_prefix_blocks = 0) and resumes: pages byte-identical to the source's, merged table = the destination
    ids, decode-step logits against the oracle."""
    s, head, lw, model = _tiny_model(kv, name, 1)
    bs = s.block_size
    ids = synth.token_ids(s, 1, n + 1)
    Kref, Vref, lref = O.forward_full(s, head, lambda l: lw[l], ids)
    nb = -(-n // bs)
    src_table = synth.block_permutation(2, 64)[:nb]
    dst_pool = synth.block_permutation(3, 64)
    dst_ids = dst_pool[:nb]
    src = kv.PagedCache(s, 64, fill=0)
    tgt = kv.PagedCache(s, 64, fill=0x5A5A)
    k = 96
    kv.kv_prefill_prefix(model, src, ids[:k], src_table[: k // bs])
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    for pos in range(k, n):
        kv.kv_decode_step(model, src, int(ids[pos]), pos, src_table[: pos // bs + 1], logits)
    wire = torch.zeros(nb * s.n_layers * 2 * (src.page_bytes // 2), dtype=torch.int16, device="cuda")
    kv.kv_pack_blocks(src, src_table, wire, wire_layout=wire_layout)
    order = np.random.default_rng(4).permutation(nb)        # blocks may arrive in any order
    if wire_layout == 0:
        page = src.page_bytes // 2
        w4 = wire.view(nb, s.n_layers * 2 * page)[torch.from_numpy(order).cuda()].contiguous().view(-1)
    else:
        w4 = wire.view(s.n_layers * 2, nb, -1)[:, torch.from_numpy(order).cuda()].contiguous().view(-1)
    merged = kv.kv_unpack_assemble(tgt, w4, order, dst_ids[order], [], n, epoch=2, expected_epoch=2,
                                   wire_layout=wire_layout)
    torch.cuda.synchronize()
    assert np.array_equal(merged, dst_ids)
    src_img, tgt_img = src.as_logical_numpy(), tgt.as_logical_numpy()
    want_status, want_merged = O.unpack_assemble(np.full_like(src_img, 0x5A5A), O.pack_blocks(src_img, src_table)[order],
                                                 order, dst_ids[order], [], n, 2, 2)
    assert want_status == O.OK and np.array_equal(want_merged, merged)
    assert np.array_equal(tgt_img[:, :, dst_ids], src_img[:, :, src_table])
    assert np.all(tgt_img[:, :, np.setdiff1d(np.arange(64), dst_ids)] == 0x5A5A)       # canaries elsewhere
    table = list(merged) + ([int(dst_pool[nb])] if n % bs == 0 else [])
    kv.kv_decode_step(model, tgt, int(ids[n]), n, table, logits)
    Kg, Vg = _kv_of(tgt, table, n + 1)
    _check_kv(s, Kg, Vg, Kref, Vref, name == "tiny", "full-copy")
    st = error_stats(logits.cpu().numpy(), lref)
    assert st["rel_l2"] <= STATED_REL_L2, st
