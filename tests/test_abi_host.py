"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol,
and rejects bad arguments before anything is enqueued (fake device addresses are never dereferenced)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import synth
from oracle import kv_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kv():
    import paper_2608_16477_b200 as kv
    kv.load()
    return kv


def test_exports_match_header(kv):
    text = open(os.path.join(ROOT, "include", "kvrebuild.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(kv_[a-z0-9_]+)\s*\(", text))
    assert declared == set(kv.EXPORTS)
    lib = kv.load()
    for name in declared:
        assert hasattr(lib, name), name


def test_status_codes_agree_with_oracle(kv):
    pairs = {"OK": 0, "ERR_ARG": -1, "ERR_SHAPE": -2, "ERR_BLOCK_RANGE": -3, "ERR_BLOCK_ALIAS": -4, "ERR_GAP": -5,
             "ERR_OVERLAP": -6, "ERR_SPLIT_UNALIGNED": -7, "ERR_TABLE_SHORT": -8, "ERR_WIRE_SIZE": -9,
             "ERR_WORKSPACE": -10, "ERR_STALE_EPOCH": -11, "ERR_TOKEN_RANGE": -12}
    text = open(os.path.join(ROOT, "include", "kvrebuild.h")).read()
    for name, val in pairs.items():
        assert getattr(O, name) == val
        assert re.search(rf"KV_{name}\s*=\s*{val}\b", text), name
        assert kv.status_string(val) != "unknown status"


def test_eq1_through_abi(kv):
    assert kv.kv_bytes_per_token(64, 8, 128, 2) == 262144 == O.kv_bytes_per_token(64, 8, 128, 2)


class _FakeCache:
    """Cache descriptor over a fake device address; only host-side validation may look at it."""

    def __init__(self, kv, shape, num_blocks, base=0x7000000000):
        from paper_2608_16477_b200.binding import CacheDesc
        page = synth.kv_page_bytes(shape)
        self.block_size = shape.block_size
        self.desc = CacheDesc(base, 2 * num_blocks * page, num_blocks * page, page, num_blocks, shape.block_size,
                              shape.n_layers, shape.n_kv_heads, shape.head_dim, 2)


class _FakeBuf:
    def __init__(self, nbytes, ptr=0x7100000000):
        self._n, self._p = nbytes, ptr

    def data_ptr(self): return self._p
    def numel(self): return self._n
    def element_size(self): return 1


def _status(fn, *a, **k):
    from paper_2608_16477_b200 import KVError
    try:
        fn(*a, **k)
    except KVError as e:
        return e.status
    return 0


def test_assemble_rejections_match_oracle(kv):
    s = synth.SHAPES["tiny"]
    cache = _FakeCache(kv, s, 12)
    page = synth.kv_page_bytes(s)
    wire = _FakeBuf(2 * s.n_layers * 2 * page)
    base = dict(logical=[2, 3], dst=[5, 6], prefix=[0, 1], n=64, epoch=3, expected=3)
    cases = [dict(epoch=2), dict(dst=[5, 12]), dict(dst=[5, -1]), dict(dst=[5, 5]), dict(dst=[5, 1]),
             dict(logical=[2, 2]), dict(logical=[1, 3]), dict(logical=[2, 4]), dict(n=65)]
    for c in cases:
        a = {**base, **c}
        want = O.check_assemble(12, s.block_size, a["logical"], a["dst"], a["prefix"], a["n"], a["epoch"], a["expected"])
        got = _status(kv.kv_unpack_assemble, cache, wire, a["logical"], a["dst"], a["prefix"], a["n"],
                      epoch=a["epoch"], expected_epoch=a["expected"], stream=0)
        assert want != 0 and got == want, (c, got, want)
    short = _FakeBuf(2 * s.n_layers * 2 * page - 16)
    assert _status(kv.kv_unpack_assemble, cache, short, [2, 3], [5, 6], [0, 1], 64, stream=0) == O.ERR_WIRE_SIZE


def test_assemble_random_defects_match_oracle(kv):
    """600 seeded argument sets (valid states with zero, one or two defects, tests/assemble_cases.py): whenever the
    oracle's check refuses a set the library refuses it with the same code, before anything is enqueued."""
    from tests.assemble_cases import random_case
    s = synth.SHAPES["tiny"]
    nb = 24
    cache = _FakeCache(kv, s, nb)
    page = synth.kv_page_bytes(s)
    refused = {}
    for seed in range(600):
        a = random_case(seed, nb, s.block_size)
        want = O.check_assemble(nb, s.block_size, a["logical"], a["dst"], a["prefix"], a["n"], a["epoch"], a["expected"])
        if want == O.OK:
            continue
        wire = _FakeBuf(max(len(a["dst"]), 1) * s.n_layers * 2 * page)
        got = _status(kv.kv_unpack_assemble, cache, wire, a["logical"], a["dst"], a["prefix"], a["n"],
                      epoch=a["epoch"], expected_epoch=a["expected"], stream=0)
        assert got == want, (seed, a, got, want)
        refused[want] = refused.get(want, 0) + 1
    assert set(refused) == {O.ERR_STALE_EPOCH, O.ERR_BLOCK_RANGE, O.ERR_BLOCK_ALIAS, O.ERR_OVERLAP, O.ERR_GAP}, refused


def test_pack_rejections(kv):
    s = synth.SHAPES["tiny"]
    cache = _FakeCache(kv, s, 12)
    page = synth.kv_page_bytes(s)
    wire = _FakeBuf(3 * s.n_layers * 2 * page)
    assert _status(kv.kv_pack_blocks, cache, [1, 12, 3], wire, stream=0) == O.ERR_BLOCK_RANGE
    assert _status(kv.kv_pack_blocks, cache, [1, 2, 3, 4], wire, stream=0) == O.ERR_WIRE_SIZE
    assert _status(kv.kv_pack_blocks, cache, [1, 2, 3], _FakeBuf(1 << 20, 0x7100000008), stream=0) == O.ERR_ARG
    assert _status(kv.kv_pack_blocks, cache, [1, 2], wire, wire_layout=5, stream=0) == O.ERR_ARG
    assert _status(kv.kv_unpack_blocks_batched, cache, [0, 2, 3], [4, 5, 4], [wire, wire], stream=0) == O.ERR_BLOCK_ALIAS


def test_prefill_and_decode_rejections(kv):
    s = synth.SHAPES["tiny"]
    lib = kv.load()
    from paper_2608_16477_b200.binding import ModelDesc, Weights
    fake = 0x7200000000
    arr = (C.c_void_p * s.n_layers)(*[fake] * s.n_layers)
    parr = C.cast(arr, C.POINTER(C.c_void_p))
    w = Weights(fake, fake, fake, parr, parr, parr, parr, parr, parr)
    d = ModelDesc(s.n_layers, s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.vocab, 1e6, 1e-6)
    h = C.c_void_p()
    assert lib.kv_model_create(C.byref(d), C.byref(w), C.byref(h)) == 0
    bad = ModelDesc(s.n_layers, s.hidden, 3, 2, s.head_dim, s.ffn, s.vocab, 1e6, 1e-6)
    h2 = C.c_void_p()
    assert lib.kv_model_create(C.byref(bad), C.byref(w), C.byref(h2)) == O.ERR_SHAPE
    # weight pointers are read as 16-byte vectors: a misaligned one is refused when the handle is created
    odd = (C.c_void_p * s.n_layers)(*[fake + 8] * s.n_layers)
    podd = C.cast(odd, C.POINTER(C.c_void_p))
    for wbad in (Weights(fake + 8, fake, fake, parr, parr, parr, parr, parr, parr),
                 Weights(fake, fake + 2, fake, parr, parr, parr, parr, parr, parr),
                 Weights(fake, fake, fake + 4, parr, parr, parr, parr, parr, parr),
                 Weights(fake, fake, fake, parr, podd, parr, parr, parr, parr),
                 Weights(fake, fake, fake, parr, parr, parr, parr, parr, podd)):
        assert lib.kv_model_create(C.byref(d), C.byref(wbad), C.byref(h2)) == O.ERR_ARG

    class M:
        handle = h
    need = kv.kv_workspace_bytes(M, kv.KV_OP_PREFILL, 64)
    assert need > 64 * s.hidden * 4
    cache = _FakeCache(kv, s, 12)
    ws = _FakeBuf(need, 0x7300000000)
    ids = list(range(64))
    table = [3, 1, 4, 5]

    def prefill(ids=ids, table=table, pos0=0, ws=ws, cache=cache):
        return _status(kv.kv_prefill_prefix, M, cache, ids, table, pos0=pos0, workspace=ws, stream=0)
    assert prefill(ids=ids[:63] + [s.vocab]) == O.ERR_TOKEN_RANGE
    assert prefill(table=[3, 1, 4]) == O.ERR_TABLE_SHORT
    assert prefill(table=[3, 1, 4, 12]) == O.ERR_BLOCK_RANGE
    assert prefill(table=[3, 1, 4, 3]) == O.ERR_BLOCK_ALIAS
    assert prefill(pos0=8, table=table + [6]) == O.ERR_SPLIT_UNALIGNED
    assert prefill(ws=_FakeBuf(need - 1, 0x7300000000)) == O.ERR_WORKSPACE
    assert prefill(ws=_FakeBuf(need, 0x7300000010)) == O.ERR_WORKSPACE
    wide = synth.ModelShape(**{**s.__dict__, "n_kv_heads": 4})
    assert prefill(cache=_FakeCache(kv, wide, 12)) == O.ERR_SHAPE
    # batched form: tables are checked per request and block ids across the whole batch
    def batched(id_lists, tabs):
        return _status(kv.kv_prefill_prefix_batched, M, cache, id_lists, tabs, workspace=ws, stream=0)
    assert batched([ids[:20], ids[:30]], [[3, 1], [4]]) == O.ERR_TABLE_SHORT        # 30 tokens need 2 blocks
    assert batched([ids[:20], ids[:30]], [[3, 1], [4, 3]]) == O.ERR_BLOCK_ALIAS     # block 3 used by both requests
    assert batched([ids[:20], ids[:30]], [[3, 1], [4, 12]]) == O.ERR_BLOCK_RANGE
    assert batched([ids[:20], [s.vocab] * 3], [[3, 1], [4]]) == O.ERR_TOKEN_RANGE
    dneed = kv.kv_workspace_bytes(M, kv.KV_OP_DECODE, 64)
    dws = _FakeBuf(dneed, 0x7300000000)
    logits = _FakeBuf(4 * s.vocab, 0x7400000000)
    assert _status(kv.kv_decode_step, M, cache, 5, 63, [3, 1, 4], logits, workspace=dws, stream=0) == O.ERR_TABLE_SHORT
    assert _status(kv.kv_decode_step, M, cache, s.vocab, 63, table, logits, workspace=dws, stream=0) == O.ERR_TOKEN_RANGE
    lib.kv_model_destroy(h)


def test_single_kernel_entry_points_reject_misaligned_arguments(kv):
    """Every vector access of the single-kernel entry points is guarded on the host: a misaligned pointer or
    descriptor returns KV_ERR_ARG and nothing is launched (the addresses here are fake and never dereferenced)."""
    from paper_2608_16477_b200.binding import CacheDesc
    lib = kv.load()
    s = synth.ModelShape("pa", n_layers=2, hidden=64, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=64, vocab=16)
    good = _FakeCache(kv, s, 16)
    page = synth.kv_page_bytes(s)
    q, out, table = 0x7500000000, 0x7500100000, 0x7500200000
    scratch = 0x7500300000
    need = kv.kv_paged_attention_scratch_bytes(8, 128, 100)

    def both(desc, q=q, out=out):
        a = lib.kv_op_paged_attention(q, 8, C.byref(desc), 0, table, 100, scratch, need, out, 0)
        b = lib.kv_op_paged_attention_noalloc(q, 8, C.byref(desc), 0, table, 100, out, 0)
        return a, b
    def desc(**kw):
        f = dict(base_dev=0x7000000000, layer_stride=2 * 16 * page, kv_stride=16 * page, block_stride=page,
                 num_blocks=16, block_size=16, n_layers=2, n_kv_heads=2, head_dim=128, elem_bytes=2)
        f.update(kw)
        return CacheDesc(*[f[n] for n, _ in CacheDesc._fields_])
    for bad in (desc(base_dev=0x7000000008), desc(layer_stride=2 * 16 * page + 8), desc(kv_stride=16 * page + 4),
                desc(block_stride=page + 2), desc(block_stride=page - 16), desc(num_blocks=0)):
        assert both(bad) == (O.ERR_ARG, O.ERR_ARG)
    assert both(desc(elem_bytes=4)) == (O.ERR_SHAPE, O.ERR_SHAPE)
    assert both(desc(head_dim=96)) == (O.ERR_SHAPE, O.ERR_SHAPE)
    assert both(good.desc, q=q + 4) == (O.ERR_ARG, O.ERR_ARG)            # q is read as float2
    assert both(good.desc, out=out + 2) == (O.ERR_ARG, O.ERR_ARG)
    assert lib.kv_op_paged_attention(q, 8, C.byref(good.desc), 0, table, 100, scratch, need - 1, out, 0) == O.ERR_WORKSPACE
    # projections: bf16 output is stored as 16-byte vectors, the residual stream updated as float4
    a, w, o, r = 0x7600000000, 0x7600100000, 0x7600200000, 0x7600300000
    for pair in (0, 0x100):
        assert lib.kv_op_gemm(a, 64, w, 32, 64, 64, 0 | pair, o + 8, None, None, 0) == O.ERR_ARG
        assert lib.kv_op_gemm(a, 64, w, 32, 64, 64, 1 | pair, None, r + 4, None, 0) == O.ERR_ARG
        assert lib.kv_op_gemm(a + 2, 64, w, 32, 64, 64, 0 | pair, o, None, None, 0) == O.ERR_ARG
        assert lib.kv_op_gemm(a, 32, w, 32, 64, 64, 0 | pair, o, None, None, 0) == O.ERR_ARG      # lda < k
        assert lib.kv_op_gemm(a, 64, w, 32, 0, 64, 0 | pair, o, None, None, 0) == O.ERR_ARG
        assert lib.kv_op_gemm(a, 64, w, 32, 60, 64, 0 | pair, o, None, None, 0) == O.ERR_SHAPE    # n not a multiple of 8
    # prefill attention: head_dim and head grouping
    assert lib.kv_op_attention_prefill(a, 10, 0, 8, 2, 96, None, 0, None, o, None, 0) == O.ERR_SHAPE
    assert lib.kv_op_attention_prefill(a, 10, 0, 7, 2, 128, None, 0, None, o, None, 0) == O.ERR_SHAPE
    assert lib.kv_op_attention_prefill(a + 8, 10, 0, 8, 2, 128, None, 0, None, o, None, 0) == O.ERR_ARG
    assert lib.kv_op_attention_prefill(a, 10, 8, 8, 2, 128, C.byref(good.desc), 0, table, o, None, 0) == O.ERR_SPLIT_UNALIGNED
    assert lib.kv_op_attention_prefill(a, 10, 16, 8, 2, 128, None, 0, table, o, None, 0) == O.ERR_ARG
    # RMSNorm reads float4 and writes four bf16 at a time; the matrix-vector product reads 16-byte vectors
    fp = lambda v: C.cast(v, C.POINTER(C.c_float))
    eps = C.c_float(1e-6)
    assert lib.kv_op_rmsnorm(fp(a + 8), w, 4, 64, eps, o, 0) == O.ERR_ARG
    assert lib.kv_op_rmsnorm(fp(a), w + 4, 4, 64, eps, o, 0) == O.ERR_ARG
    assert lib.kv_op_rmsnorm(fp(a), w, 4, 64, eps, o + 4, 0) == O.ERR_ARG
    assert lib.kv_op_rmsnorm(fp(a), w, 4, 66, eps, o, 0) == O.ERR_ARG
    assert lib.kv_op_gemv(w + 8, fp(a), 16, 64, 0, None, eps, fp(r), 0) == O.ERR_ARG
    assert lib.kv_op_gemv(w, fp(a + 4), 16, 64, 0, None, eps, fp(r), 0) == O.ERR_ARG
    assert lib.kv_op_gemv(w, fp(a), 16, 60, 0, None, eps, fp(r), 0) == O.ERR_SHAPE


def test_gemm_plan_query(kv):
    """The launcher's choice is a pure function of the problem size and the SM count (148 assumed without a device)."""
    pair, bn = kv.kv_gemm_plan(128, 5120, 1)
    assert pair is False and bn in (128, 160, 192, 224, 256)
    pair, bn = kv.kv_gemm_plan(4096, 10240, 3, head_dim=128)
    assert pair is True and bn % 128 == 0
    pair, bn = kv.kv_gemm_plan(4096, 25600, 2)
    assert pair is True and bn % 64 == 0
    from paper_2608_16477_b200 import KVError
    with pytest.raises(KVError):
        kv.kv_gemm_plan(4096, 10240, 3, head_dim=96)
    with pytest.raises(KVError):
        kv.kv_gemm_plan(0, 10240, 1)


def test_header_is_plain_c_and_a_c_program_links(kv, tmp_path):
    """The header compiles as strict C99 (no C++, no torch types) and a C program linked against the library runs the
    host-only entry points."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    assert gcc, "gcc is part of the build environment"
    libdir = os.path.dirname(kv.lib_path())
    exe = str(tmp_path / "abi_c_consumer")
    subprocess.run([gcc, "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I" + os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "abi_c_consumer.c"), "-o", exe, "-L" + libdir, "-lkvrebuild",
                    "-Wl,-rpath," + libdir], check=True, capture_output=True, text=True)
    run = subprocess.run([exe], capture_output=True, text=True)
    assert run.returncode == 0, (run.returncode, run.stdout, run.stderr)
    assert run.stdout.startswith("t_w=")
