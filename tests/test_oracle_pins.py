"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU)."""
import math
import os

import numpy as np
import pytest

import synth
from oracle import kv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- Eq. (1)
def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "eq1_kv_footprint.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_eq1_printed_values():
    rows = _golden_rows()
    L, H, d, b, expect = map(int, rows[0])
    assert O.kv_bytes_per_token(L, H, d, b) == expect == 262144
    assert O.kv_bytes_per_token(L, H, d, b) == int(rows[1][0]) * 1024
    tokens, gib, mbps, secs = rows[2]
    total = O.kv_bytes(int(tokens), L, H, d, b)
    assert total == 1_048_576_000
    assert abs(total / 2**30 - float(gib)) < 0.03           # "approximately 1 GiB"
    assert abs(total * 8 / (float(mbps) * 1e6) - float(secs)) < 0.1   # "approximately 28 seconds"
    assert O.kv_bytes(4096, L, H, d, b) == 2**30


def test_eq1_matches_page_geometry():
    # bytes per token summed over all pages of the paged image equal Eq. (1)
    for name, expect in (("tiny", 1024), ("8b", 147456), ("32b", 262144)):
        s = synth.SHAPES[name]
        assert O.kv_bytes_per_token(s.n_layers, s.n_kv_heads, s.head_dim) == expect
        assert 2 * s.n_layers * synth.kv_page_bytes(s) == expect * s.block_size
    c = O.new_cache(3, 5, 16, 2, 8)
    assert c.nbytes == 5 * 16 * O.kv_bytes_per_token(3, 2, 8)


# ---------------------------------------------------------------- bf16 image
def test_bf16_rounding_matches_library():
    torch = pytest.importorskip("torch")
    r = np.random.default_rng(0)
    x = np.concatenate([r.standard_normal(50000) * 10 ** r.uniform(-6, 6, 50000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 65280.0]]).astype(np.float32)
    want = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.to_bf16_bits(x), want)
    assert np.array_equal(O.from_bf16_bits(want), torch.tensor(x).to(torch.bfloat16).float().numpy())


# ---------------------------------------------------------------- RMSNorm
def test_rmsnorm_hand_vector():
    x = np.array([[1.0, 2.0, 3.0, 4.0]])
    g = np.array([2.0, 1.0, 0.5, 1.0])
    want = np.array([[2.0, 2.0, 1.5, 4.0]]) / math.sqrt(7.5)
    assert np.allclose(O.rmsnorm(x, g, 0.0), want, rtol=0, atol=1e-15)
    # eps sits inside the square root
    assert np.allclose(O.rmsnorm(x, g, 2.5), np.array([[2.0, 2.0, 1.5, 4.0]]) / math.sqrt(10.0), atol=1e-15)


def test_rmsnorm_unit_rms_and_scale_invariance():
    r = np.random.default_rng(1)
    x = r.standard_normal((7, 64)) * 3.0
    y = O.rmsnorm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt(np.mean(y * y, axis=-1)), 1.0, atol=1e-14)
    assert np.allclose(O.rmsnorm(5.0 * x, np.ones(64), 0.0), y, atol=1e-14)
    # rows are normalised independently
    assert np.allclose(O.rmsnorm(x[2:3], np.ones(64), 0.0), y[2:3], atol=0)


# ---------------------------------------------------------------- RoPE
def test_rope_identity_norm_and_explicit_angles():
    r = np.random.default_rng(2)
    x = r.standard_normal((6, 3, 8))
    assert np.array_equal(O.rope(x, np.zeros(6), 1e6), x)
    y = O.rope(x, np.arange(6) + 11, 1e6)
    assert np.allclose(x[..., :4] ** 2 + x[..., 4:] ** 2, y[..., :4] ** 2 + y[..., 4:] ** 2, atol=1e-13)
    # d = 4, base 10000: theta = [1, 1/100]; unit vector on the first pair turns by pos radians
    e = np.zeros((1, 1, 4)); e[0, 0, 0] = 1.0
    out = O.rope(e, np.array([3]), 1e4)[0, 0]
    assert np.allclose(out, [math.cos(3.0), 0.0, math.sin(3.0), 0.0], atol=1e-15)
    e = np.zeros((1, 1, 4)); e[0, 0, 3] = 1.0       # second pair's "b" component, theta_1 = 0.01
    out = O.rope(e, np.array([50]), 1e4)[0, 0]
    assert np.allclose(out, [0.0, -math.sin(0.5), 0.0, math.cos(0.5)], atol=1e-15)


def test_rope_relative_position_property():
    r = np.random.default_rng(3)
    q = r.standard_normal((1, 1, 64)); k = r.standard_normal((1, 1, 64))
    def dot(m, n):
        return float(np.sum(O.rope(q, np.array([m]), 1e6) * O.rope(k, np.array([n]), 1e6)))
    assert abs(dot(17, 5) - dot(17 + 1000, 5 + 1000)) < 1e-9
    assert abs(dot(17, 5) - dot(12, 0)) < 1e-9
    assert abs(dot(17, 5) - dot(5, 17)) > 1e-3      # not symmetric: sign of the rotation matters


# ---------------------------------------------------------------- SwiGLU
def test_silu_closed_forms():
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert abs(O.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16
    assert abs(O.silu(np.array([40.0]))[0] - 40.0) < 1e-12
    assert abs(O.silu(np.array([-40.0]))[0]) < 1e-12
    assert abs(O.silu(np.array([-1.0]))[0] + 1.0 / (1.0 + math.e)) < 1e-16


# ---------------------------------------------------------------- attention
def _attention_loops(q, k, v, q_pos0=0):
    tq, hq, d = q.shape
    tk, hkv, _ = k.shape
    out = np.zeros((tq, hq, d))
    for i in range(tq):
        for h in range(hq):
            g = h // (hq // hkv)
            scores = []
            for j in range(tk):
                if j <= q_pos0 + i:
                    scores.append(sum(q[i, h, c] * k[j, g, c] for c in range(d)) / math.sqrt(d))
            m = max(scores)
            e = [math.exp(s - m) for s in scores]
            z = sum(e)
            for j, ej in enumerate(e):
                for c in range(d):
                    out[i, h, c] += ej / z * v[j, g, c]
    return out


def test_attention_bruteforce_loops():
    r = np.random.default_rng(4)
    q = r.standard_normal((5, 4, 6)); k = r.standard_normal((5, 2, 6)); v = r.standard_normal((5, 2, 6))
    assert np.allclose(O.attention(q, k, v), _attention_loops(q, k, v), atol=1e-13)
    # continued rows: 2 new queries at positions 3, 4 over 5 keys
    assert np.allclose(O.attention(q[3:], k, v, q_pos0=3), _attention_loops(q, k, v)[3:], atol=1e-13)


def test_attention_special_cases():
    r = np.random.default_rng(5)
    q = r.standard_normal((9, 4, 8)); k = r.standard_normal((9, 2, 8)); v = r.standard_normal((9, 2, 8))
    o = O.attention(q, k, v)
    assert np.allclose(o[0, 0], v[0, 0]) and np.allclose(o[0, 3], v[0, 1])      # row 0 sees key 0 only
    const = np.broadcast_to(np.array([1.5, -2.0, 0.25, 3.0, 0, 0, 1, 2.0]), v.shape)
    assert np.allclose(O.attention(q, k, const), np.broadcast_to(const[0, 0], q.shape), atol=1e-13)
    # GQA == MHA over replicated KV heads
    assert np.allclose(o, O.attention(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1)), atol=1e-14)
    # future keys do not matter
    k2, v2 = k.copy(), v.copy(); k2[6:] += 5.0; v2[6:] -= 3.0
    assert np.array_equal(O.attention(q, k2, v2)[:6], o[:6])


def test_attention_vs_library_sdpa():
    torch = pytest.importorskip("torch")
    r = np.random.default_rng(6)
    q = r.standard_normal((33, 4, 16)); k = r.standard_normal((33, 2, 16)); v = r.standard_normal((33, 2, 16))
    tq = torch.tensor(q).permute(1, 0, 2)[None]
    tk = torch.tensor(np.repeat(k, 2, axis=1)).permute(1, 0, 2)[None]
    tv = torch.tensor(np.repeat(v, 2, axis=1)).permute(1, 0, 2)[None]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.allclose(O.attention(q, k, v), want, atol=1e-12)


# ---------------------------------------------------------------- projections
def test_projection_orientation_and_layout():
    # y = x W^T with W [out, in]; Q | K | V row order; gate | up row order: use one-hot weights
    s = synth.ModelShape("t", n_layers=1, hidden=8, n_q_heads=2, n_kv_heads=1, head_dim=4, ffn=8, vocab=5)
    w = {"attn_norm": np.ones(8), "ffn_norm": np.ones(8),
         "w_qkv": np.zeros((16, 8)), "w_o": np.zeros((8, 8)),
         "w_gate_up": np.zeros((16, 8)), "w_down": np.zeros((8, 8))}
    # K head reads hidden[0:4], V head reads hidden[4:8]
    for c in range(4):
        w["w_qkv"][8 + c, c] = 1.0
        w["w_qkv"][12 + c, 4 + c] = 1.0
    x = np.arange(1.0, 9.0)[None, :]
    _, k, v = O.layer_forward(s, w, x, np.array([0]))
    h = x / math.sqrt(np.mean(x * x) + s.rms_eps)
    assert np.allclose(k[0, 0], h[0, :4]) and np.allclose(v[0, 0], h[0, 4:])
    got = O._mm(np.array([[1.0, 2.0]]), np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]), np.float64)
    assert np.array_equal(got, [[1.0, 2.0, 3.0]])


def test_layer_identity_weights_pass_through():
    # attention with one token returns V; identity projections make every stage checkable by hand
    s = synth.ModelShape("t", n_layers=1, hidden=4, n_q_heads=1, n_kv_heads=1, head_dim=4, ffn=4, vocab=3,
                         rms_eps=0.0)
    eye = np.eye(4)
    w = {"attn_norm": np.ones(4), "ffn_norm": np.ones(4), "w_qkv": np.vstack([eye, eye, eye]), "w_o": eye,
         "w_gate_up": np.vstack([eye, eye]), "w_down": eye}
    x = np.array([[2.0, -2.0, 2.0, -2.0]])
    x1, k, v = O.layer_forward(s, w, x, np.array([0]))
    h = x / 2.0                               # rms = 2
    assert np.allclose(v[0, 0], h[0]) and np.allclose(k[0, 0], h[0])
    x_mid = x + h                             # single key: o = v
    h2 = x_mid / 3.0                          # rms of (3,-3,3,-3)
    want = x_mid + (h2 / (1 + np.exp(-h2))) * h2
    assert np.allclose(x1, want, atol=1e-14)


def test_whole_model_vs_library_llama():
    """Black-box cross-check of the complete forward on the tiny shapes against a randomly
    initialised library decoder loaded with the same weights (fp32 CPU)."""
    torch = pytest.importorskip("torch")
    tf = pytest.importorskip("transformers")
    s = synth.SHAPES["tiny-sharp"]
    cfg = tf.LlamaConfig(vocab_size=s.vocab, hidden_size=s.hidden, intermediate_size=s.ffn,
                         num_hidden_layers=s.n_layers, num_attention_heads=s.n_q_heads,
                         num_key_value_heads=s.n_kv_heads, head_dim=s.head_dim, rms_norm_eps=s.rms_eps,
                         rope_theta=s.rope_base, attention_bias=False, mlp_bias=False,
                         tie_word_embeddings=False, max_position_embeddings=512,
                         attn_implementation="eager")
    try:
        cfg.rope_parameters = {"rope_type": "default", "rope_theta": s.rope_base}
    except Exception:
        pass
    model = tf.LlamaForCausalLM(cfg).float().eval()
    head = synth.head_weights(s, 0)
    layers = [synth.layer_weights(s, 0, l) for l in range(s.n_layers)]
    qd, kd = s.q_dim, s.kv_dim
    sd = {"model.embed_tokens.weight": head["embed"], "model.norm.weight": head["final_norm"],
          "lm_head.weight": head["lm_head"]}
    for l, w in enumerate(layers):
        p = f"model.layers.{l}."
        sd[p + "input_layernorm.weight"] = w["attn_norm"]
        sd[p + "post_attention_layernorm.weight"] = w["ffn_norm"]
        sd[p + "self_attn.q_proj.weight"] = w["w_qkv"][:qd]
        sd[p + "self_attn.k_proj.weight"] = w["w_qkv"][qd:qd + kd]
        sd[p + "self_attn.v_proj.weight"] = w["w_qkv"][qd + kd:]
        sd[p + "self_attn.o_proj.weight"] = w["w_o"]
        sd[p + "mlp.gate_proj.weight"] = w["w_gate_up"][:s.ffn]
        sd[p + "mlp.up_proj.weight"] = w["w_gate_up"][s.ffn:]
        sd[p + "mlp.down_proj.weight"] = w["w_down"]
    missing = model.load_state_dict({k: torch.tensor(np.array(v)) for k, v in sd.items()}, strict=False)
    assert not [m for m in missing.missing_keys if "rotary" not in m]
    ids = synth.token_ids(s, 0, 40)
    with torch.no_grad():
        out = model(torch.tensor(ids[None].astype(np.int64)), use_cache=True)
    K, V, logits = O.forward_full(s, head, lambda l: layers[l], ids, all_logits=True)
    want = out.logits[0].numpy()
    assert np.max(np.abs(logits - want)) < 2e-3 * max(1.0, np.max(np.abs(want)))
    pkv = out.past_key_values
    for l in range(s.n_layers):
        try:
            kl, vl = pkv.layers[l].keys, pkv.layers[l].values
        except AttributeError:
            kl, vl = pkv[l][0], pkv[l][1]
        assert np.allclose(K[l], kl[0].permute(1, 0, 2).numpy(), atol=2e-4)
        assert np.allclose(V[l], vl[0].permute(1, 0, 2).numpy(), atol=2e-4)


# ---------------------------------------------------------------- causality
@pytest.mark.parametrize("name", ["tiny", "tiny-sharp"])
def test_prefix_plus_incremental_equals_full(name):
    s = synth.SHAPES[name]
    head = synth.head_weights(s, 0)
    lw = [synth.layer_weights(s, 0, l) for l in range(s.n_layers)]
    layers = lambda l: lw[l]
    k_split, n = 32, 41
    ids = synth.token_ids(s, 0, n + 1)
    Kf, Vf, logits_f = O.forward_full(s, head, layers, ids)                 # positions 0..n
    Kp, Vp, _ = O.forward_full(s, head, layers, ids[:k_split], want_logits=False)
    assert np.allclose(Kp, Kf[:, :k_split], rtol=0, atol=1e-10 * np.max(np.abs(Kf)))
    assert np.allclose(Vp, Vf[:, :k_split], rtol=0, atol=1e-10 * np.max(np.abs(Vf)))
    Kc = np.zeros_like(Kf); Vc = np.zeros_like(Vf)
    Kc[:, :k_split], Vc[:, :k_split] = Kp, Vp
    for pos in range(k_split, n + 1):
        kn, vn, lg = O.decode_step(s, head, layers, ids[pos], pos, Kc, Vc)
        Kc[:, pos], Vc[:, pos] = kn, vn
    assert np.max(np.abs(Kc - Kf)) <= 1e-5 * np.max(np.abs(Kf))
    assert np.max(np.abs(Vc - Vf)) <= 1e-5 * np.max(np.abs(Vf))
    assert np.max(np.abs(lg - logits_f)) <= 1e-5 * np.max(np.abs(logits_f))


def test_future_tokens_do_not_change_past_kv():
    s = synth.SHAPES["tiny-sharp"]
    head = synth.head_weights(s, 0)
    lw = [synth.layer_weights(s, 0, l) for l in range(s.n_layers)]
    ids = synth.token_ids(s, 0, 24)
    K0, V0, _ = O.forward_full(s, head, lambda l: lw[l], ids)
    ids2 = ids.copy(); ids2[17] = (ids2[17] + 1) % s.vocab
    K1, V1, _ = O.forward_full(s, head, lambda l: lw[l], ids2)
    assert np.allclose(K0[:, :17], K1[:, :17], rtol=0, atol=1e-12) and np.allclose(V0[:, :17], V1[:, :17], rtol=0, atol=1e-12)
    assert not np.allclose(K0[:, 17:], K1[:, 17:])


# ---------------------------------------------------------------- pack / unpack / assemble
def _random_cache(seed, L=3, nb=12, bs=4, hkv=2, d=4):
    bits = np.random.default_rng(seed).integers(0, 65536, (L, 2, nb, bs, hkv, d)).astype(np.uint16)
    return bits


def test_pack_five_deep_byte_loop():
    c = _random_cache(0)
    ids = [7, 2, 9]
    wire = O.pack_blocks(c, ids)
    cb = c.view(np.uint8).reshape(3, 2, 12, -1)           # bytes of each page
    wb = wire.view(np.uint8).reshape(-1)
    page_bytes = cb.shape[-1]
    pos = 0
    for i, b in enumerate(ids):                           # wire order: block, layer, K/V, page bytes
        for l in range(3):
            for kv in range(2):
                for byte in range(page_bytes):
                    assert wb[pos] == cb[l, kv, b, byte]
                    pos += 1
    assert pos == wb.size


def test_pack_identity_and_permutation():
    c = _random_cache(1)
    all_ids = list(range(12))
    # block-major view of the cache: packing ids 0..m-1 is a plain transpose-copy
    assert np.array_equal(O.pack_blocks(c, all_ids), c.transpose(2, 0, 1, 3, 4, 5).reshape(12, 3, 2, -1))
    perm = np.random.default_rng(2).permutation(12)
    assert np.array_equal(O.pack_blocks(c, perm), O.pack_blocks(c, all_ids)[perm])


def test_unpack_roundtrip_canary_and_table():
    src = _random_cache(3)
    ids = [5, 1, 8]
    wire = O.pack_blocks(src, ids)
    dst = np.full_like(src, 0xBEEF)
    st, merged = O.unpack_assemble(dst, wire, logical=[3, 2, 4], dst_ids=[10, 0, 6], prefix_table=[4, 9],
                                   n_tokens_total=5 * 4 - 1)
    assert st == O.OK
    assert list(merged) == [4, 9, 0, 10, 6]              # prefix table, then dst ids in logical order
    for i, (s_id, d_id) in enumerate(zip(ids, [10, 0, 6])):
        assert np.array_equal(dst[:, :, d_id], src[:, :, s_id])
    untouched = [b for b in range(12) if b not in (10, 0, 6)]
    assert np.all(dst[:, :, untouched] == 0xBEEF)
    # NaN payloads / -0 / denormals survive: bytes are copied as integers
    assert dst.dtype == np.uint16


def test_assemble_checks():
    src = _random_cache(4)
    wire = O.pack_blocks(src, [1, 2])
    def run(**kw):
        a = dict(logical=[2, 3], dst_ids=[5, 6], prefix_table=[0, 1], n_tokens_total=16, epoch=3, expected_epoch=3)
        a.update(kw)
        dst = np.zeros_like(src)
        st, merged = O.unpack_assemble(dst, wire, **a)
        if st != O.OK:
            assert merged is None and not dst.any()          # destination untouched on error
        return st
    assert run() == O.OK
    assert run(epoch=2) == O.ERR_STALE_EPOCH
    assert run(dst_ids=[5, 12]) == O.ERR_BLOCK_RANGE
    assert run(dst_ids=[5, -1]) == O.ERR_BLOCK_RANGE
    assert run(dst_ids=[5, 5]) == O.ERR_BLOCK_ALIAS
    assert run(dst_ids=[5, 1]) == O.ERR_BLOCK_ALIAS          # collides with a prefix block
    assert run(logical=[2, 2]) == O.ERR_OVERLAP
    assert run(logical=[1, 3]) == O.ERR_OVERLAP              # lands inside the prefix
    assert run(logical=[2, 4]) == O.ERR_OVERLAP              # beyond ceil(n / Bs)
    assert run(n_tokens_total=17) == O.ERR_GAP               # needs logical block 4 as well
    assert run(n_tokens_total=13) == O.OK                    # partial last block is a full page


def test_write_read_kv_through_block_table():
    L, nb, bs, hkv, d = 2, 8, 4, 2, 4
    c = O.new_cache(L, nb, bs, hkv, d)
    r = np.random.default_rng(5)
    K = r.standard_normal((L, 10, hkv, d)); V = r.standard_normal((L, 10, hkv, d))
    table = [6, 0, 3]
    O.write_kv(c, K, V, table)
    # position 5 -> block table[1] = 0, slot 1
    assert np.array_equal(c[1, 0, 0, 1], O.to_bf16_bits(K[1, 5]))
    assert np.array_equal(c[0, 1, 3, 1], O.to_bf16_bits(V[0, 9]))
    k2, v2 = O.read_kv(c, table, 10)
    assert np.array_equal(k2, O.from_bf16_bits(O.to_bf16_bits(K)))
    assert np.array_equal(v2, O.from_bf16_bits(O.to_bf16_bits(V)))
    assert not c[:, :, [1, 2, 4, 5, 7]].any()


def test_bf16_storage_points_only_round():
    """The bf16-storage variant is the same function with roundings inserted: its K/V are exactly
    bf16-representable, it stays within a few bf16 ulps of the exact path, and on inputs where every
    stored tensor is already representable it changes nothing."""
    s = synth.SHAPES["tiny"]
    head = synth.head_weights(s, 0)
    lw = [synth.layer_weights(s, 0, l) for l in range(s.n_layers)]
    ids = synth.token_ids(s, 0, 48)
    K0, V0, l0 = O.forward_full(s, head, lambda l: lw[l], ids)
    K1, V1, l1 = O.forward_full(s, head, lambda l: lw[l], ids, act_bf16=True)
    assert np.array_equal(K1, O.from_bf16_bits(O.to_bf16_bits(K1))) and np.array_equal(V1, O.from_bf16_bits(O.to_bf16_bits(V1)))
    assert 0 < np.max(np.abs(K1 - K0)) < 2e-2 and np.sqrt(np.sum((l1 - l0) ** 2) / np.sum(l0 ** 2)) < 1e-2
    # powers of two everywhere: nothing to round
    t = synth.ModelShape("t", n_layers=1, hidden=4, n_q_heads=1, n_kv_heads=1, head_dim=4, ffn=4, vocab=3, rms_eps=0.0)
    eye = np.eye(4)
    w = {"attn_norm": np.ones(4), "ffn_norm": np.ones(4), "w_qkv": np.vstack([eye, eye, eye]), "w_o": eye,
         "w_gate_up": np.vstack([eye, eye]), "w_down": eye}
    x = np.array([[2.0, -2.0, 2.0, -2.0]])
    a = O.layer_forward(t, w, x, np.array([0]), skip_after_kv=True)
    b = O.layer_forward(t, w, x, np.array([0]), skip_after_kv=True, act_bf16=True)
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])


# ---------------------------------------------------------------- continued (chunked) prefill
@pytest.mark.parametrize("name", ["tiny", "tiny-sharp"])
@pytest.mark.parametrize("chunks", [(16,) * 6, (48, 48), (33, 1, 47, 15), (96,)])
def test_chunked_prefill_equals_full(name, chunks):
    """Chunk-by-chunk evaluation over a cached prefix (k_past / v_past) is the same function as the
    single-pass forward: every chunk size, ragged splits and a one-token chunk included."""
    s = synth.SHAPES[name]
    head = synth.head_weights(s, 0)
    lw = [synth.layer_weights(s, 0, l) for l in range(s.n_layers)]
    ids = synth.token_ids(s, 0, sum(chunks))
    Kf, Vf, lf = O.forward_full(s, head, lambda l: lw[l], ids)
    Kc, Vc, lc = O.forward_chunked(s, head, lambda l: lw[l], ids, chunks)
    for got, want in ((Kc, Kf), (Vc, Vf), (lc, lf)):
        assert got.shape == want.shape
        assert np.max(np.abs(got - want)) <= 1e-10 * np.max(np.abs(want))
    # K/V-only form: the last layer of the last chunk stops after its K/V, same values
    Kn, Vn, ln = O.forward_chunked(s, head, lambda l: lw[l], ids, chunks, want_logits=False)
    assert ln is None and np.array_equal(Kn, Kc) and np.array_equal(Vn, Vc)


def test_chunked_prefill_past_is_used_and_ordered():
    """A wrong past must show: dropping the cached prefix, or pairing its keys with the wrong values, changes the
    chunk's output (reordering keys and values together does not: every past position is visible to every
    row of the chunk, and the positions are already rotated into the keys)."""
    s = synth.SHAPES["tiny-sharp"]
    w = synth.layer_weights(s, 0, 0)
    r = np.random.default_rng(3)
    x = r.standard_normal((40, s.hidden))
    xa, ka, va = O.layer_forward(s, w, x[:24], np.arange(24))
    xb, kb, vb = O.layer_forward(s, w, x[24:], np.arange(24, 40), k_past=ka, v_past=va)
    xf, kf, vf = O.layer_forward(s, w, x, np.arange(40))
    assert np.allclose(np.concatenate([xa, xb]), xf, rtol=0, atol=1e-11 * np.max(np.abs(xf)))
    assert np.allclose(np.concatenate([ka, kb]), kf, rtol=0, atol=1e-12)
    x_nopast, _, _ = O.layer_forward(s, w, x[24:], np.arange(24, 40))
    x_rev, _, _ = O.layer_forward(s, w, x[24:], np.arange(24, 40), k_past=ka[::-1], v_past=va[::-1])
    x_mix, _, _ = O.layer_forward(s, w, x[24:], np.arange(24, 40), k_past=ka[::-1], v_past=va)
    assert np.max(np.abs(x_nopast - xb)) > 1e-3 and np.max(np.abs(x_mix - xb)) > 1e-3
    assert np.max(np.abs(x_rev - xb)) <= 1e-11 * np.max(np.abs(xb))
    # K and V of the new rows never depend on the past
    _, k2, v2 = O.layer_forward(s, w, x[24:], np.arange(24, 40), skip_after_kv=True)
    assert np.array_equal(k2, kb) and np.array_equal(v2, vb)


# ---------------------------------------------------------------- fp32 library matmul (used on the largest shapes)
def test_fp32_matmul_against_fp64_and_error_bound():
    r = np.random.default_rng(8)
    x = synth.bf16_round_f32(r.standard_normal((256, 384), dtype=np.float32))
    w = synth.bf16_round_f32(r.standard_normal((512, 384), dtype=np.float32) * np.float32(0.05))
    exact = O._mm(x, w, np.float64)
    got = O._mm(x, w, np.float32)
    assert got.dtype == np.float64 and got.shape == (256, 512)
    assert np.sqrt(np.sum((got - exact) ** 2) / np.sum(exact ** 2)) <= 1e-5
    # textbook bound for a length-k fp32 dot product in any summation order: |err| <= k u sum|x||w| (u = 2^-24),
    # plus the final rounding of the result
    k, u = 384, 2.0 ** -24
    bound = (k + 1) * u * (np.abs(x).astype(np.float64) @ np.abs(w).astype(np.float64).T)
    assert np.all(np.abs(got - exact) <= bound)
    # orientation: y = x W^T
    assert np.array_equal(O._mm(np.eye(3), np.arange(6.0).reshape(2, 3), np.float32), np.arange(6.0).reshape(2, 3).T)


def test_fp32_matmul_forward_tracks_fp64_forward():
    s = synth.SHAPES["tiny-sharp"]
    head = synth.head_weights(s, 0)
    lw = [synth.layer_weights(s, 0, l) for l in range(s.n_layers)]
    ids = synth.token_ids(s, 0, 64)
    K0, V0, l0 = O.forward_full(s, head, lambda l: lw[l], ids)
    K1, V1, l1 = O.forward_full(s, head, lambda l: lw[l], ids, mm_dtype=np.float32)
    for a, b in ((K1, K0), (V1, V0), (l1, l0)):
        assert np.sqrt(np.sum((a - b) ** 2) / np.sum(b ** 2)) <= 1e-5


# ---------------------------------------------------------------- bf16 storage points, one by one
def test_bf16_storage_points_against_library_casts():
    """Where the storage-precision evaluation rounds: one layer restated with library tensor ops in fp64 and a
    library bfloat16 cast at each of the tensors a 16-bit pipeline keeps between contractions (normed input,
    post-RoPE Q and K, V, attention output, normed FFN input, SwiGLU output) and nowhere else (the residual
    stream, scores, probabilities and accumulators stay wide)."""
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    s = synth.SHAPES["tiny-sharp"]
    w = synth.layer_weights(s, 0, 1)
    r = np.random.default_rng(12)
    t = 24
    x = r.standard_normal((t, s.hidden)) * 1.7
    pos = np.arange(5, 5 + t)
    kp = synth.bf16_round_f32(r.standard_normal((5, s.n_kv_heads, s.head_dim), dtype=np.float32))
    vp = synth.bf16_round_f32(r.standard_normal((5, s.n_kv_heads, s.head_dim), dtype=np.float32))
    got_x, got_k, got_v = O.layer_forward(s, w, x, pos, k_past=kp, v_past=vp, act_bf16=True)

    def cast(a):
        return a.to(torch.bfloat16).to(torch.float64)

    def norm(a, g):
        return a * torch.rsqrt((a * a).mean(-1, keepdim=True) + s.rms_eps) * g

    def rot(a):     # [T, H, d]
        half = s.head_dim // 2
        inv = torch.tensor([s.rope_base ** (-2.0 * j / s.head_dim) for j in range(half)], dtype=torch.float64)
        ang = torch.tensor(pos, dtype=torch.float64)[:, None] * inv[None]
        c, sn = torch.cos(ang)[:, None], torch.sin(ang)[:, None]
        a1, a2 = a[..., :half], a[..., half:]
        return torch.cat([a1 * c - a2 * sn, a2 * c + a1 * sn], -1)

    W = {k: torch.tensor(np.asarray(v), dtype=torch.float64) for k, v in w.items()}
    xt = torch.tensor(x)
    h = cast(norm(xt, W["attn_norm"]))
    qkv = h @ W["w_qkv"].T
    hq, hkv, d = s.n_q_heads, s.n_kv_heads, s.head_dim
    q = cast(rot(qkv[:, : hq * d].reshape(t, hq, d)))
    k = cast(rot(qkv[:, hq * d: (hq + hkv) * d].reshape(t, hkv, d)))
    v = cast(qkv[:, (hq + hkv) * d:].reshape(t, hkv, d))
    k_all = torch.cat([torch.tensor(kp, dtype=torch.float64), k]).repeat_interleave(hq // hkv, dim=1)
    v_all = torch.cat([torch.tensor(vp, dtype=torch.float64), v]).repeat_interleave(hq // hkv, dim=1)
    mask = torch.arange(5 + t)[None, :] <= torch.tensor(pos)[:, None]
    o = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None], k_all.permute(1, 0, 2)[None],
                                       v_all.permute(1, 0, 2)[None], attn_mask=mask)[0].permute(1, 0, 2)
    x1 = xt + cast(o).reshape(t, hq * d) @ W["w_o"].T
    h2 = cast(norm(x1, W["ffn_norm"]))
    ab = h2 @ W["w_gate_up"].T
    m = cast(F.silu(ab[:, : s.ffn]) * ab[:, s.ffn:])
    x2 = x1 + m @ W["w_down"].T
    assert np.array_equal(got_k, k.numpy()) or np.max(np.abs(got_k - k.numpy())) <= 2.0 ** -7 * np.max(np.abs(got_k))
    # identical rounding decisions except where a pre-rounding value sits within fp64 noise of a tie
    assert np.mean(got_k != k.numpy()) < 1e-3 and np.mean(got_v != v.numpy()) < 1e-3
    assert np.max(np.abs(got_x - x2.numpy())) <= 1e-9 * np.max(np.abs(got_x))
    # and the roundings matter: the exact layer differs by far more than the agreement above
    ex_x, _, _ = O.layer_forward(s, w, x, pos, k_past=kp, v_past=vp)
    assert np.max(np.abs(ex_x - got_x)) > 1e-4
