"""Parity of the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

import synth
from oracle import kv_oracle as O
from tests.scenario import error_stats, oracle_reference, oracle_reference_bf16_storage, run_gpu_scenario

pytestmark = pytest.mark.gpu

# stated tolerance for bf16 K/V and next-token logits against the oracle
MAX_ABS = 2e-2
REL_L2 = 1e-2


@pytest.fixture(scope="module")
def kv():
    import paper_2608_16477_b200 as kv
    kv.load()
    return kv


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _bits_to_torch(torch, bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


# ------------------------------------------------------------------ pack / unpack: bit exact
@pytest.mark.parametrize("cache_layout", ["layer_major", "block_major"])
@pytest.mark.parametrize("wire_layout", [0, 1])
def test_pack_unpack_bit_exact_tiny(kv, torch, cache_layout, wire_layout):
    s = synth.SHAPES["tiny"]
    nb = 64
    rng = np.random.default_rng(10)
    img = rng.integers(0, 65536, (s.n_layers, 2, nb, s.block_size, s.n_kv_heads, s.head_dim)).astype(np.uint16)
    src = kv.PagedCache(s, nb, layout=cache_layout)
    page = src.page_bytes // 2
    flat = img.reshape(s.n_layers, 2, nb, page)
    src.data.copy_(_bits_to_torch(torch, flat if cache_layout == "layer_major" else flat.transpose(2, 0, 1, 3)))
    ids = synth.block_permutation(1, nb)[:10]
    wire = torch.zeros(10 * s.n_layers * 2 * page, dtype=torch.int16, device="cuda")
    kv.kv_pack_blocks(src, ids, wire, wire_layout=wire_layout)
    want = O.pack_blocks(img, ids)                                     # [i, L, 2, page]
    if wire_layout == 1:
        want = want.transpose(1, 2, 0, 3)
    assert np.array_equal(wire.cpu().numpy().view(np.uint16), want.reshape(-1))
    # unpack into a canary-filled cache
    dst = kv.PagedCache(s, nb, layout=cache_layout, fill=0x5A5A)
    dst_img = np.full_like(img, 0x5A5A)
    dst_ids = synth.block_permutation(2, nb)[8:18]
    prefix = synth.block_permutation(2, nb)[:8]
    merged = kv.kv_unpack_assemble(dst, wire, np.arange(8, 18), dst_ids, prefix, 18 * s.block_size - 3,
                                   wire_layout=wire_layout)
    st, want_merged = O.unpack_assemble(dst_img, O.pack_blocks(img, ids), np.arange(8, 18), dst_ids, prefix,
                                        18 * s.block_size - 3)
    assert st == O.OK and np.array_equal(merged, want_merged)
    assert np.array_equal(dst.as_logical_numpy(), dst_img)             # pages and canaries, whole cache


def test_unpack_assemble_random_cases_against_oracle(kv, torch):
    """300 seeded migration states (tests/assemble_cases.py: arbitrary arrival order, partly filled last block, empty
    prefix or empty suffix, and defects of every kind the consistency checks exist for): status, merged table and
    the whole cache image equal the oracle's, bit for bit; a refused set leaves the cache untouched."""
    from paper_2608_16477_b200 import KVError
    from tests.assemble_cases import random_case
    s = synth.SHAPES["tiny"]
    nb = 24
    page = synth.kv_page_bytes(s) // 2
    rng = np.random.default_rng(77)
    dst = kv.PagedCache(s, nb, fill=0x5A5A)
    want_img = np.full((s.n_layers, 2, nb, s.block_size, s.n_kv_heads, s.head_dim), 0x5A5A, dtype=np.uint16)
    accepted = 0
    for seed in range(300):
        a = random_case(seed, nb, s.block_size)
        n_wire = len(a["dst"])
        wire_np = rng.integers(0, 65536, (max(n_wire, 1), s.n_layers, 2, page)).astype(np.uint16)
        wire = _bits_to_torch(torch, wire_np)
        want_st, want_merged = O.unpack_assemble(want_img, wire_np[:n_wire].reshape(n_wire, s.n_layers, 2, s.block_size,
                                                                                    s.n_kv_heads, s.head_dim),
                                                 a["logical"], a["dst"], a["prefix"], a["n"], a["epoch"], a["expected"])
        try:
            merged = kv.kv_unpack_assemble(dst, wire, a["logical"], a["dst"], a["prefix"], a["n"], epoch=a["epoch"],
                                           expected_epoch=a["expected"], wire_bytes=n_wire * s.n_layers * 2 * page * 2)
            got_st = 0
        except KVError as e:
            got_st, merged = e.status, None
        assert got_st == want_st, (seed, a, got_st, want_st)
        if want_st == O.OK:
            accepted += 1
            assert np.array_equal(merged, want_merged), (seed, a)
        assert np.array_equal(dst.as_logical_numpy(), want_img), (seed, a)
    kv.kv_check_copy_status()
    assert accepted >= 60


def test_pack_ragged_and_empty(kv, torch):
    # odd geometry: page of 1 slot x 1 head x 32 dims = 64 bytes; more blocks than one launch carries
    s = synth.ModelShape("odd", n_layers=3, hidden=64, n_q_heads=1, n_kv_heads=1, head_dim=32, ffn=64, vocab=16,
                         block_size=1)
    nb = 2500
    rng = np.random.default_rng(11)
    img = rng.integers(0, 65536, (3, 2, nb, 1, 1, 32)).astype(np.uint16)
    src = kv.PagedCache(s, nb)
    src.data.copy_(_bits_to_torch(torch, img.reshape(3, 2, nb, 32)))
    ids = synth.block_permutation(3, nb)[:2001]                        # 3 launches of <= 960 ids
    wire = torch.zeros(2001 * 3 * 2 * 32, dtype=torch.int16, device="cuda")
    kv.kv_pack_blocks(src, ids, wire)
    assert np.array_equal(wire.cpu().numpy().view(np.uint16), O.pack_blocks(img, ids).reshape(-1))
    kv.kv_pack_blocks(src, [], wire)                                   # empty list: no-op
    dst = kv.PagedCache(s, nb, fill=0)
    merged = kv.kv_unpack_assemble(dst, wire, np.arange(2001), ids[::-1].copy(), [], 2001)
    assert np.array_equal(merged, ids[::-1])
    want = np.zeros_like(img)
    want[:, :, ids[::-1]] = img[:, :, ids]
    assert np.array_equal(dst.as_logical_numpy(), want)


def test_pack_unpack_beyond_one_parameter_block(kv, torch):
    """More blocks (9,001) than one launch's parameter block carries (7,680) in a single request, and more requests
    (70) than it has records for (64) in a batched call: the lists continue in further launches, a request may
    straddle two of them, and every page still lands where the oracle puts it."""
    s = synth.ModelShape("odd", n_layers=2, hidden=64, n_q_heads=1, n_kv_heads=1, head_dim=32, ffn=64, vocab=16,
                         block_size=1)
    nb = 9100
    rng = np.random.default_rng(13)
    img = rng.integers(0, 65536, (2, 2, nb, 1, 1, 32)).astype(np.uint16)
    src = kv.PagedCache(s, nb)
    src.data.copy_(_bits_to_torch(torch, img.reshape(2, 2, nb, 32)))
    ids = synth.block_permutation(14, nb)[:9001]
    for layout in (0, 1):
        wire = torch.zeros(9001 * 2 * 2 * 32, dtype=torch.int16, device="cuda")
        kv.kv_pack_blocks(src, ids, wire, wire_layout=layout)
        want = O.pack_blocks(img, ids)
        if layout == 1:
            want = want.transpose(1, 2, 0, 3)
        assert np.array_equal(wire.cpu().numpy().view(np.uint16), want.reshape(-1)), layout
    # 70 requests of 1..9 blocks each through the batched calls
    counts = [1 + (i * 7) % 9 for i in range(70)]
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    rid = synth.block_permutation(15, nb)[: offs[-1]]
    wires = [torch.zeros(c * 2 * 2 * 32, dtype=torch.int16, device="cuda") for c in counts]
    kv.kv_pack_blocks_batched(src, offs, rid, wires)
    for r, c in enumerate(counts):
        want = O.pack_blocks(img, rid[offs[r]:offs[r + 1]])
        assert np.array_equal(wires[r].cpu().numpy().view(np.uint16), want.reshape(-1)), r
    dst = kv.PagedCache(s, nb, fill=0)
    did = synth.block_permutation(16, nb)[: offs[-1]]
    kv.kv_unpack_blocks_batched(dst, offs, did, wires)
    want_img = np.zeros_like(img)
    want_img[:, :, did] = img[:, :, rid]
    assert np.array_equal(dst.as_logical_numpy(), want_img)
    kv.kv_check_copy_status()


def test_pack_unpack_batched_pattern_32b_pages(kv, torch):
    """32 KiB pages, 64 layers: a scaled-down form of the 16-request stress workload whose content is the
    counter-based pattern, checked page by page against the host generator."""
    s = synth.SHAPES["32b"]
    nb_src, nb_dst = 192, 160
    src = kv.PagedCache(s, nb_src)
    total = src.data.numel() * 2
    kv.kv_fill_pattern(src.data, total, seed=99)
    counts = [max(1, c // 16) for c in synth.STRESS_BLOCK_COUNTS[:6]]   # 27, 21, 18, 11, 12, 5
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    src_ids = synth.block_permutation(5, nb_src)[: offs[-1]]
    dst_ids = synth.block_permutation(6, nb_dst)[: offs[-1]]
    page = src.page_bytes
    wires = [torch.empty(c * s.n_layers * 2 * page, dtype=torch.uint8, device="cuda") for c in counts]
    kv.kv_pack_blocks_batched(src, offs, src_ids, wires)
    dst = kv.PagedCache(s, nb_dst, fill=0)
    kv.kv_unpack_blocks_batched(dst, offs, dst_ids, wires)
    torch.cuda.synchronize()
    rng = np.random.default_rng(7)
    for _ in range(40):                                                # sampled pages, oracle one by one
        r = int(rng.integers(0, len(counts)))
        i = int(rng.integers(0, counts[r]))
        l = int(rng.integers(0, s.n_layers)); kvi = int(rng.integers(0, 2))
        b_src = int(src_ids[offs[r] + i]); b_dst = int(dst_ids[offs[r] + i])
        src_off = ((l * 2 + kvi) * nb_src + b_src) * page
        want = synth.pattern_bytes(99, src_off, page)
        w_off = ((i * s.n_layers + l) * 2 + kvi) * page
        assert np.array_equal(wires[r][w_off:w_off + page].cpu().numpy(), want)
        got = dst.data[l, kvi, b_dst].cpu().numpy().view(np.uint8)
        assert np.array_equal(got, want)
    # everything outside the destination ids is still zero
    mask = np.ones(nb_dst, dtype=bool); mask[dst_ids] = False
    assert not dst.data[:, :, torch.from_numpy(np.nonzero(mask)[0]).cuda()].any()


# ------------------------------------------------------------------ single kernels
@pytest.mark.parametrize("m,n,k", [(128, 256, 64), (300, 520, 192), (1000, 1048, 512), (16, 8, 64), (257, 1280, 1024),
                                   (512, 25600, 256), (512, 4736, 128), (1024, 12288, 64)])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_gemm_tensor_core(kv, torch, m, n, k, mode):
    rng = np.random.default_rng(100 + m + n + k + mode)
    a = synth.bf16_round_f32(rng.standard_normal((m, k), dtype=np.float32))
    rows = 2 * n if mode == 2 else n
    w = synth.bf16_round_f32(rng.standard_normal((rows, k), dtype=np.float32) / np.float32(np.sqrt(k)))
    ref = a.astype(np.float64) @ w.astype(np.float64).T
    ta = torch.from_numpy(a).cuda().to(torch.bfloat16)
    tw = torch.from_numpy(w).cuda().to(torch.bfloat16)
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    if mode == 1:
        r0 = rng.standard_normal((m, n), dtype=np.float32)
        resid = torch.from_numpy(r0).cuda()
        kv.kv_op_gemm(ta, tw, 1, resid=resid, status=status)
        got = resid.cpu().numpy()
        want = r0 + ref
        tol = 1e-4 * np.sqrt(k) / 8
    else:
        out = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device="cuda")
        kv.kv_op_gemm(ta, tw, mode, out=out, status=status)
        got = out.float().cpu().numpy()
        want = ref if mode == 0 else O.silu(ref[:, :n]) * ref[:, n:]
        tol = None
    torch.cuda.synchronize()
    assert int(status[0]) == 0, f"device wait ran out: {status[:8].tolist()}"
    if tol is None:       # bf16 output: half an ulp relative plus fp32 accumulation noise
        assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-3), error_stats(got, want)
    else:
        assert np.max(np.abs(got - want)) <= tol, error_stats(got, want)


@pytest.mark.parametrize("m,n,k", [(129, 520, 192), (256, 256, 64), (300, 520, 192), (1000, 1048, 512), (4096, 5120, 256)])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_gemm_cta_pair_identical_to_single_cta(kv, torch, m, n, k, mode):
    """The cta_group::2 kernel (two SMs per 256-row tile) accumulates in the same order as the one-CTA kernel."""
    g = torch.Generator(device="cuda").manual_seed(m + n + k + mode)
    a = torch.empty(m, k, dtype=torch.bfloat16, device="cuda").normal_(0.0, 1.0, generator=g)
    w = torch.empty(2 * n if mode == 2 else n, k, dtype=torch.bfloat16, device="cuda").normal_(0.0, 0.05, generator=g)
    r0 = torch.randn(m, n, device="cuda", generator=g)
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    res = []
    for flag in (0, 0x100):
        out = torch.zeros(m, n, dtype=torch.bfloat16, device="cuda")
        resid = r0.clone()
        kv.kv_op_gemm(a, w, mode | flag, out=None if mode == 1 else out, resid=resid if mode == 1 else None,
                      status=status, n=n)
        torch.cuda.synchronize()
        res.append(resid if mode == 1 else out)
    assert int(status[0]) == 0, status[:8].tolist()
    assert torch.equal(res[0], res[1])
    assert bool(res[0].float().abs().sum() > 0)


# (14400, 64): enough row pairs to fill the SMs with warps (the lighter four-loads-in-flight form of the kernel);
# the other cases run the form with eight loads in flight per row and lane
@pytest.mark.parametrize("n,k", [(37, 256), (512, 5120), (1001, 1064), (14400, 64), (300, 2056)])
@pytest.mark.parametrize("mode,norm", [(0, False), (0, True), (1, False), (2, False), (2, True)])
def test_gemv_decode(kv, torch, n, k, mode, norm):
    rng = np.random.default_rng(n + k + mode)
    rows = 2 * n if mode == 2 else n
    w = synth.bf16_round_f32(rng.standard_normal((rows, k), dtype=np.float32) / np.float32(np.sqrt(k)))
    x = (rng.standard_normal(k) * 2.0).astype(np.float32)
    g = synth.bf16_round_f32(rng.uniform(0.5, 1.5, k).astype(np.float32))
    y0 = rng.standard_normal(n).astype(np.float32)
    xin = O.rmsnorm(x[None], g, 1e-6)[0] if norm else x.astype(np.float64)
    prod = w.astype(np.float64) @ xin
    want = prod if mode == 0 else (y0 + prod if mode == 1 else O.silu(prod[:n]) * prod[n:])
    y = torch.from_numpy(y0.copy()).cuda()
    kv.kv_op_gemv(torch.from_numpy(w).cuda().to(torch.bfloat16), torch.from_numpy(x).cuda(), mode, y,
                  gain=torch.from_numpy(g).cuda().to(torch.bfloat16) if norm else None, eps=1e-6)
    got = y.cpu().numpy()
    assert np.max(np.abs(got - want)) <= 2e-5 * np.sqrt(k) * max(1.0, np.max(np.abs(want))), error_stats(got, want)


def test_rmsnorm_rows(kv, torch):
    rng = np.random.default_rng(6)
    x = (rng.standard_normal((37, 5120)) * 3).astype(np.float32)
    g = synth.bf16_round_f32(rng.uniform(0.5, 1.5, 5120).astype(np.float32))
    out = torch.empty(37, 5120, dtype=torch.bfloat16, device="cuda")
    kv.kv_op_rmsnorm(torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda().to(torch.bfloat16), 1e-6, out)
    want = O.rmsnorm(x, g, 1e-6)
    got = out.float().cpu().numpy()
    assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-6)


# the last two cases give the persistent kernel more work items than SMs: 200 items (a partial second round,
# walked backwards) and 300 items (two full rounds and a partial third) on 148 SMs
# (100, 6, 2, 128) and (300, 3, 1, 64): an odd number of query heads per KV head (the last head of a group is
# paired with itself); (129, 2, 2, 128): one query head per KV head
@pytest.mark.parametrize("t,hq,hkv,d", [(70, 4, 2, 64), (200, 8, 1, 128), (129, 2, 2, 128), (1000, 4, 2, 128),
                                      (384, 8, 2, 64), (128, 2, 1, 128), (1, 2, 1, 64), (6400, 8, 2, 64),
                                      (3200, 24, 4, 64), (100, 6, 2, 128), (300, 3, 1, 64)])
def test_attention_prefill_kernel(kv, torch, t, hq, hkv, d):
    rng = np.random.default_rng(7 + t)
    qkv = synth.bf16_round_f32(rng.standard_normal((t, (hq + 2 * hkv) * d), dtype=np.float32))
    q = qkv[:, : hq * d].reshape(t, hq, d)
    k = qkv[:, hq * d: (hq + hkv) * d].reshape(t, hkv, d)
    v = qkv[:, (hq + hkv) * d:].reshape(t, hkv, d)
    want = O.attention(q, k, v)
    out = torch.empty(t, hq * d, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    kv.kv_op_attention_prefill(torch.from_numpy(qkv).cuda().to(torch.bfloat16), hq, hkv, d, out, status=status)
    got = out.float().cpu().numpy().reshape(t, hq, d)
    assert int(status[0]) == 0
    st = error_stats(got, want)
    assert st["max_abs"] <= MAX_ABS and st["rel_l2"] <= REL_L2, st


@pytest.mark.parametrize("pos0,t,hq,hkv,d", [(48, 80, 4, 2, 64), (256, 200, 6, 2, 128), (16, 1, 2, 1, 128)])
def test_attention_prefill_kernel_over_cached_prefix(kv, torch, pos0, t, hq, hkv, d):
    """The single-kernel entry point with pos0 > 0: the K/V of positions [0, pos0) come from pages of a cache (through a
    fragmented block table), the chunk's rows from the qkv buffer; against the oracle's attention over the whole context."""
    s = synth.ModelShape("ap", n_layers=2, hidden=64, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, ffn=64, vocab=16)
    rng = np.random.default_rng(70 + pos0)
    n_ctx = pos0 + t
    qkv = synth.bf16_round_f32(rng.standard_normal((n_ctx, (hq + 2 * hkv) * d), dtype=np.float32))
    q = qkv[:, : hq * d].reshape(n_ctx, hq, d)
    k = qkv[:, hq * d: (hq + hkv) * d].reshape(n_ctx, hkv, d)
    v = qkv[:, (hq + hkv) * d:].reshape(n_ctx, hkv, d)
    want = O.attention(q[pos0:], k, v, q_pos0=pos0)
    nb = 64
    table = synth.block_permutation(12, nb)[: pos0 // 16]
    img = O.new_cache(2, nb, 16, hkv, d)
    kk = np.zeros((2, pos0, hkv, d)); vv = np.zeros((2, pos0, hkv, d))
    kk[1], vv[1] = k[:pos0], v[:pos0]
    O.write_kv(img, kk, vv, table)
    cache = kv.PagedCache(s, nb)
    cache.data.copy_(_bits_to_torch(torch, img.reshape(2, 2, nb, -1)))
    buf = torch.from_numpy(qkv).cuda().to(torch.bfloat16)
    buf[:pos0] = 7.0                                   # the call must fetch the prefix's K/V itself
    out = torch.empty(t, hq * d, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    kv.kv_op_attention_prefill(buf, hq, hkv, d, out, pos0=pos0, cache=cache, layer=1,
                               block_table_dev=torch.from_numpy(table).cuda(), status=status)
    got = out.float().cpu().numpy().reshape(t, hq, d)
    assert int(status[0]) == 0
    st = error_stats(got, want)
    assert st["max_abs"] <= MAX_ABS and st["rel_l2"] <= REL_L2, st


@pytest.mark.parametrize("scale", [4.0, 12.0])
def test_attention_prefill_kernel_wide_score_range(kv, torch, scale):
    """Scores with a standard deviation of 16 and 144 instead of 1: running maxima that jump by far more than the lazy
    rescaling threshold, exponents far below the clamp of the FMA-pipe exponential (2^-126), rows dominated by a single
    key.  Every exponential path (special-function unit, polynomial, masked) must agree with the oracle."""
    t, hq, hkv, d = 700, 4, 2, 128
    rng = np.random.default_rng(int(scale) + 40)
    qkv = rng.standard_normal((t, (hq + 2 * hkv) * d), dtype=np.float32)
    qkv[:, : (hq + hkv) * d] *= np.float32(scale)                    # queries and keys
    qkv = synth.bf16_round_f32(qkv)
    q = qkv[:, : hq * d].reshape(t, hq, d)
    k = qkv[:, hq * d: (hq + hkv) * d].reshape(t, hkv, d)
    v = qkv[:, (hq + hkv) * d:].reshape(t, hkv, d)
    want = O.attention(q, k, v)
    out = torch.empty(t, hq * d, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    kv.kv_op_attention_prefill(torch.from_numpy(qkv).cuda().to(torch.bfloat16), hq, hkv, d, out, status=status)
    got = out.float().cpu().numpy().reshape(t, hq, d)
    assert int(status[0]) == 0 and np.all(np.isfinite(got))
    st = error_stats(got, want)
    assert st["max_abs"] <= MAX_ABS and st["rel_l2"] <= REL_L2, st


def test_attention_prefill_long_context_sampled_rows(kv, torch):
    """8,192 tokens (64 key tiles for the last row tile, 256 work items on 148 SMs): three windows of query rows are
    checked against the oracle, which scores each window against the keys up to its last row."""
    t, hq, hkv, d = 8192, 8, 2, 128
    rng = np.random.default_rng(99)
    qkv = synth.bf16_round_f32(rng.standard_normal((t, (hq + 2 * hkv) * d), dtype=np.float32))
    out = torch.empty(t, hq * d, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    kv.kv_op_attention_prefill(torch.from_numpy(qkv).cuda().to(torch.bfloat16), hq, hkv, d, out, status=status)
    assert int(status[0]) == 0
    got = out.float().cpu().numpy().reshape(t, hq, d)
    q = qkv[:, : hq * d].reshape(t, hq, d)
    k = qkv[:, hq * d: (hq + hkv) * d].reshape(t, hkv, d)
    v = qkv[:, (hq + hkv) * d:].reshape(t, hkv, d)
    for r0, r1 in ((0, 130), (4030, 4170), (8060, 8192)):
        want = O.attention(q[r0:r1], k[:r1], v[:r1], q_pos0=r0)
        st = error_stats(got[r0:r1], want)
        assert st["max_abs"] <= MAX_ABS and st["rel_l2"] <= REL_L2, (r0, st)


@pytest.mark.parametrize("n_ctx,hq,hkv,d,ramp", [
    (777, 8, 2, 128, 0), (1, 4, 2, 64, 0), (128, 16, 1, 128, 0), (129, 8, 1, 64, 0), (300, 40, 1, 128, 0),
    (4609, 64, 8, 128, 0), (20011, 8, 1, 128, 0),
    # more 128-key tiles than the grid has parts (two CTAs per SM over the KV heads): a CTA walks several tiles with a
    # running maximum; `ramp` makes the scores grow (+) or shrink (-) along the context so that maximum keeps moving
    (4737, 16, 8, 128, 0), (9000, 16, 8, 128, 3), (20011, 32, 8, 64, -3), (7000, 160, 8, 64, 2), (33000, 8, 4, 128, 1)])
def test_paged_decode_attention(kv, torch, n_ctx, hq, hkv, d, ramp):
    """One query position against a paged context: a single key, exactly one 128-key split, one key past it, many
    splits, several tiles per CTA; groups of 2 to 40 query heads per KV head (more than the 16 rows one pass of the
    kernel serves)."""
    s = synth.ModelShape("pa", n_layers=2, hidden=64, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, ffn=64, vocab=16)
    nb = -(-n_ctx // 16) + 7
    rng = np.random.default_rng(8 + n_ctx)
    K = rng.standard_normal((2, n_ctx, hkv, d), dtype=np.float32)
    if ramp:
        pos = np.arange(n_ctx, dtype=np.float32) / n_ctx
        K *= (1.0 + abs(ramp) * (pos if ramp > 0 else 1.0 - pos))[None, :, None, None]
    K = synth.bf16_round_f32(K)
    V = synth.bf16_round_f32(rng.standard_normal((2, n_ctx, hkv, d), dtype=np.float32))
    img = O.new_cache(2, nb, 16, hkv, d)
    table = synth.block_permutation(9, nb)[: -(-n_ctx // 16)]
    O.write_kv(img, K, V, table)
    cache = kv.PagedCache(s, nb)
    cache.data.copy_(_bits_to_torch(torch, img.reshape(2, 2, nb, -1)))
    q = rng.standard_normal((hq, d)).astype(np.float32)
    want = O.attention(q[None], K[1], V[1], q_pos0=n_ctx - 1)[0]
    scratch = torch.empty(kv.kv_paged_attention_scratch_bytes(hq, d, n_ctx), dtype=torch.uint8, device="cuda")
    out = torch.empty(hq, d, dtype=torch.float32, device="cuda")
    kv.kv_op_paged_attention(torch.from_numpy(q).cuda(), cache, 1, torch.from_numpy(table).cuda(), n_ctx, scratch, out)
    assert np.max(np.abs(out.cpu().numpy() - want)) < 1e-4


# ------------------------------------------------------------------ whole path
def _check_scenario(shape, res, Kref, Vref, logits_ref, n, literal):
    assert np.array_equal(res["merged"], res["expected_merged"])
    # wire and destination pages are byte-identical to the source pages
    want_wire = O.pack_blocks(res["src_img"], res["src_suffix_ids"])
    assert np.array_equal(res["wire"], want_wire.reshape(-1))
    for s_id, d_id in zip(res["src_suffix_ids"], res["dst_ids"]):
        assert np.array_equal(res["tgt_after_unpack"][:, :, d_id], res["src_img"][:, :, s_id])
    report = {}
    for name, got, ref in (("K", res["K"], Kref), ("V", res["V"], Vref), ("logits", res["logits"], logits_ref)):
        st = error_stats(got, ref)
        report[name] = st
        assert st["rel_l2"] <= REL_L2, (name, st)
        if literal:
            assert st["max_abs"] <= MAX_ABS, (name, st)
        else:
            assert st["scaled_ok"], (name, st)
    print(shape.name, report)
    return report


@pytest.mark.parametrize("name", ["tiny", "tiny-sharp"])
@pytest.mark.parametrize("n_suffix", [32, 37])
def test_scenario_tiny(kv, name, n_suffix):
    s = synth.SHAPES[name]
    k, n = 128, 128 + n_suffix
    ids = synth.token_ids(s, 0, n + 1)
    Kref, Vref, logits_ref = oracle_reference(s, 0, ids)
    res = run_gpu_scenario(kv, s, 0, ids, k, n)
    _check_scenario(s, res, Kref, Vref, logits_ref, n, literal=(name == "tiny"))
    # prefill logits = oracle logits of the prefix's last row
    _, _, lp = oracle_reference(s, 0, ids[:k])
    st = error_stats(res["prefill_logits"], lp)
    assert st["rel_l2"] <= REL_L2, st


def test_scenario_odd_query_group(kv):
    """Three query heads per KV head (an odd group: the prefill attention pairs the third head with itself) and one
    query head per KV head, through the whole path against the oracle."""
    for hq, hkv in ((6, 2), (2, 2)):
        s = synth.ModelShape(f"odd{hq}", n_layers=2, hidden=192, n_q_heads=hq, n_kv_heads=hkv, head_dim=64, ffn=384,
                             vocab=512, sharp=True)
        ids = synth.token_ids(s, 0, 150)
        Kref, Vref, logits_ref = oracle_reference(s, 0, ids)
        res = run_gpu_scenario(kv, s, 0, ids, 112, 149)
        assert np.array_equal(res["merged"], res["expected_merged"])
        for name, got, ref in (("K", res["K"], Kref), ("V", res["V"], Vref), ("logits", res["logits"], logits_ref)):
            st = error_stats(got, ref)
            assert st["rel_l2"] <= REL_L2 and st["scaled_ok"], (hq, name, st)
        _, _, lp = oracle_reference(s, 0, ids[:112])
        assert error_stats(res["prefill_logits"], lp)["rel_l2"] <= REL_L2


@pytest.mark.parametrize("dims", [
    dict(hidden=264, n_q_heads=6, n_kv_heads=3, head_dim=64, ffn=520, vocab=1001),     # nothing a multiple of a tile
    dict(hidden=136, n_q_heads=3, n_kv_heads=3, head_dim=128, ffn=200, vocab=333),     # one query head per KV head, d 128
    dict(hidden=72, n_q_heads=10, n_kv_heads=2, head_dim=64, ffn=40, vocab=50),        # five heads per group, tiny widths
])
def test_scenario_awkward_dimensions(kv, dims):
    """Model dimensions that are multiples of 8 (the interface's only requirement) and of no tile size: every kernel's
    ragged column and K tails, through the whole path against the oracle (prefix 208 = 13 blocks, resume at 300: above
    one 128-row tile, a partly filled last block)."""
    s = synth.ModelShape("awkward", n_layers=2, sharp=True, **dims)
    ids = synth.token_ids(s, 3, 301)
    Kref, Vref, logits_ref = oracle_reference(s, 3, ids)
    res = run_gpu_scenario(kv, s, 3, ids, 208, 300)
    assert np.array_equal(res["merged"], res["expected_merged"])
    for name, got, ref in (("K", res["K"], Kref), ("V", res["V"], Vref), ("logits", res["logits"], logits_ref)):
        st = error_stats(got, ref)
        assert st["rel_l2"] <= REL_L2 and st["scaled_ok"], (dims, name, st)
    _, _, lp = oracle_reference(s, 3, ids[:208])
    assert error_stats(res["prefill_logits"], lp)["rel_l2"] <= REL_L2


def test_scenario_tiny_block_major_layer_major_wire(kv):
    s = synth.SHAPES["tiny-sharp"]
    ids = synth.token_ids(s, 0, 161)
    Kref, Vref, logits_ref = oracle_reference(s, 0, ids)
    res = run_gpu_scenario(kv, s, 0, ids, 128, 160, cache_layout="block_major", wire_layout=1)
    assert np.array_equal(res["merged"], res["expected_merged"])
    for name, got, ref in (("K", res["K"], Kref), ("V", res["V"], Vref), ("logits", res["logits"], logits_ref)):
        st = error_stats(got, ref)
        assert st["rel_l2"] <= REL_L2 and st["scaled_ok"], (name, st)


@pytest.mark.parametrize("name,layers,k,n", [("8b", 2, 512, 560), ("32b", 2, 1024, 1064)])
def test_scenario_wide_reduced_depth(kv, name, layers, k, n):
    """Full-width shapes at reduced depth (the oracle finishes in about a minute).

    Two comparisons.  (1) Against the oracle evaluated at the pipeline's bf16 storage points: what remains
    is accumulation order and the ulp flips it causes downstream, so the bound is tighter than the stated one.  (2) Against the exact oracle: the
    stated relative-L2 bound; max-abs is checked in the scaled form because K/V values beyond |4| have a
    bf16 half-ulp of 0.0156 and more, so no two-byte cache can meet a literal 2e-2 on every element."""
    s = synth.SHAPES[name].with_layers(layers)
    s = synth.ModelShape(**{**s.__dict__, "vocab": 4096})
    ids = synth.token_ids(s, 0, n + 1)
    res = run_gpu_scenario(kv, s, 0, ids, k, n, num_blocks=128)
    assert np.array_equal(res["merged"], res["expected_merged"])
    Ke, Ve, le = oracle_reference_bf16_storage(s, 0, ids, k)
    report = {}
    for nm, got, ref in (("K", res["K"], Ke), ("V", res["V"], Ve), ("logits", res["logits"], le)):
        st = error_stats(got, ref)
        report["bf16pt_" + nm] = st
        assert st["rel_l2"] <= 5e-3, (nm, st)                      # half the stated bound
        # element-wise: the rel-L2 bound caps the error's standard deviation at 5e-3 * rms(ref); 8 sigma
        # covers ~1e9 roughly Gaussian samples, plus one bf16 ulp of the value itself (at most 2^-7 |ref|)
        rms = float(np.sqrt(np.mean(np.asarray(ref, dtype=np.float64) ** 2)))
        assert np.all(np.abs(got - ref) <= 8 * 5e-3 * rms + 2.0 ** -7 * np.abs(ref)), (nm, st)
    Kref, Vref, logits_ref = oracle_reference(s, 0, ids)
    for nm, got, ref in (("K", res["K"], Kref), ("V", res["V"], Vref)):
        st = error_stats(got, ref)
        report["exact_" + nm] = st
        assert st["rel_l2"] <= REL_L2, (nm, st)
    report["exact_logits"] = error_stats(res["logits"], logits_ref)
    assert report["exact_logits"]["rel_l2"] <= 2 * REL_L2, report["exact_logits"]
    print(s.name, report)


def test_chunked_prefill_matches_single_shot(kv, torch):
    s = synth.SHAPES["tiny-sharp"]
    ids = synth.token_ids(s, 3, 160)
    head = synth.head_weights(s, 3)
    model = kv.Model(s, head, lambda l: synth.layer_weights(s, 3, l))
    table = synth.block_permutation(4, 64)[:10]
    one = kv.PagedCache(s, 64, fill=0)
    two = kv.PagedCache(s, 64, fill=0)
    kv.kv_prefill_prefix(model, one, ids, table)
    kv.kv_prefill_prefix(model, two, ids[:64], table[:4])
    kv.kv_prefill_prefix(model, two, ids[64:], table, pos0=64)
    torch.cuda.synchronize()
    a = O.from_bf16_bits(one.as_logical_numpy()).astype(np.float64)
    b = O.from_bf16_bits(two.as_logical_numpy()).astype(np.float64)
    st = error_stats(b, a)
    assert st["rel_l2"] <= 5e-3, st


def test_chunked_prefill_wide_shape_tensor_core_path(kv, torch):
    """Continued prefill in 256-token chunks (the chunk size the paper uses under contention, Section 6.3) on a
    32B-shaped two-layer model: the cached prefix is gathered for the tensor-core attention kernel.  The result
    must agree with the single-shot prefill up to the ulp flips a different tile split of the same sums causes."""
    s = synth.SHAPES["32b"].with_layers(2)
    s = synth.ModelShape(**{**s.__dict__, "vocab": 2048})
    n = 1000                                           # ragged: last chunk has 232 tokens
    ids = synth.token_ids(s, 5, n)
    head = synth.head_weights(s, 5)
    model = kv.Model(s, head, lambda l: synth.layer_weights(s, 5, l))
    table = synth.block_permutation(6, 128)[: -(-n // 16)]
    one = kv.PagedCache(s, 128, fill=0)
    two = kv.PagedCache(s, 128, fill=0)
    lg1 = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    lg2 = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    ws = kv.kv_prefill_prefix(model, one, ids, table, logits_out=lg1)
    kv.kv_check_device_status(ws)
    for p0 in range(0, n, 256):
        chunk = ids[p0:p0 + 256]
        last = p0 + 256 >= n
        ws = kv.kv_prefill_prefix(model, two, chunk, table[: -(-(p0 + len(chunk)) // 16)], pos0=p0,
                                  logits_out=lg2 if last else None)
        kv.kv_check_device_status(ws)
    torch.cuda.synchronize()
    a = O.from_bf16_bits(one.as_logical_numpy()).astype(np.float64)
    b = O.from_bf16_bits(two.as_logical_numpy()).astype(np.float64)
    st = error_stats(b, a)
    sl = error_stats(lg2.cpu().numpy(), lg1.cpu().numpy())
    print("chunked vs single-shot:", st, sl)
    assert st["rel_l2"] <= 5e-3 and sl["rel_l2"] <= 1e-2, (st, sl)


@pytest.mark.parametrize("name,layers,lengths", [("tiny-sharp", 2, (100, 37, 260)), ("32b", 2, (512, 300))])
def test_batched_prefill_equals_separate_calls(kv, torch, name, layers, lengths):
    """Several prefix reconstructions in one call: every page and the per-request logits must be identical to
    separate calls (rows of a projection do not depend on the other rows in the launch; attention runs per request)."""
    s = synth.SHAPES[name].with_layers(layers)
    s = synth.ModelShape(**{**s.__dict__, "vocab": min(s.vocab, 2048)})
    head = synth.head_weights(s, 9)
    model = kv.Model(s, head, lambda l: synth.layer_weights(s, 9, l))
    perm = synth.block_permutation(10, 256)
    ids, tables, used = [], [], 0
    for i, n in enumerate(lengths):
        ids.append(synth.token_ids(s, 20 + i, n))
        nb = -(-n // s.block_size)
        tables.append(perm[used:used + nb].copy())
        used += nb
    one = kv.PagedCache(s, 256, fill=0)
    two = kv.PagedCache(s, 256, fill=0)
    lg_sep = torch.zeros(len(lengths), s.vocab, dtype=torch.float32, device="cuda")
    lg_bat = torch.zeros_like(lg_sep)
    for i in range(len(lengths)):
        ws = kv.kv_prefill_prefix(model, one, ids[i], tables[i], logits_out=lg_sep[i])
        kv.kv_check_device_status(ws)
    ws = kv.kv_prefill_prefix_batched(model, two, ids, tables, logits_out=lg_bat)
    kv.kv_check_device_status(ws)
    torch.cuda.synchronize()
    assert torch.equal(one.data, two.data)
    assert bool(one.data.any())
    assert torch.equal(lg_sep, lg_bat)
    # K/V-only form (last layer stops after its K/V): same pages
    three = kv.PagedCache(s, 256, fill=0)
    kv.kv_prefill_prefix_batched(model, three, ids, tables)
    torch.cuda.synchronize()
    assert torch.equal(one.data, three.data)


# ------------------------------------------------------------------ failure detection on the device
def test_bounded_wait_gives_up_and_reports(kv, torch):
    """Every wait inside the tensor-core kernels is bounded.  The self-test kernel makes one run out on purpose (a
    barrier that nothing signals, a 200 us limit): the wait records itself in the status block, the other threads
    leave through the CTA's abort flag, the kernel returns, the host reads KV_ERR_DEVICE, and the context is intact:
    the next operation on the same workspace runs and reports a clean status."""
    s = synth.SHAPES["tiny"]
    head = synth.head_weights(s, 0)
    model = kv.Model(s, head, lambda l: synth.layer_weights(s, 0, l))
    ws = model.workspace(kv.KV_OP_PREFILL, 64)
    kv.kv_selftest_bounded_wait(ws, 200)
    with pytest.raises(kv.KVError) as e:
        kv.kv_check_device_status(ws)
    assert e.value.status == -14                                   # KV_ERR_DEVICE
    words = ws[:32].view(torch.int32).tolist()                     # error, tag, detail[0..5]
    assert words[0] == -14 and words[1] == 99 and words[2] == 0 and words[3] == 0
    assert words[5] == 64                                          # every thread's wait was abandoned, one recorded
    cache = kv.PagedCache(s, 16, fill=0)
    kv.kv_prefill_prefix(model, cache, synth.token_ids(s, 0, 64), [3, 1, 4, 5], workspace=ws)
    kv.kv_check_device_status(ws)                                  # clean again
    assert bool(cache.data.any())
