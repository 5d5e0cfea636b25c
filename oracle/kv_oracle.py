"""CPU oracle for target-side KV-cache reconstruction.  TEST INFRASTRUCTURE ONLY.

A plain, slow, deliberately unoptimised numpy implementation (fp64 arithmetic unless a
caller asks for fp32 matmuls on the largest shapes) of what the hot path computes:

  * prefill of a stable prefix by a decoder-only GQA transformer and the K/V it leaves in a
    paged block cache (the paper's "Initialization and parallel preparation": the target
    reconstructs the prefix KV cache through local prefill from the exact prefix token ids);
  * one incremental decoding step on a cache (source-side suffix production and the target's
    resume at position n, "Final synchronization and activation");
  * extraction of suffix blocks into a contiguous wire buffer (Section 5, "Parallel state
    preparation": physical block ids -> per-layer KV tensors -> bytes);
  * scatter of those blocks into freshly allocated pages and assembly of the merged block
    table, with the state-consistency checks of Section 4.3 ("State consistency").

The paper never fixes the model internals (it runs stock checkpoints); the architecture here
is the standard pre-norm GQA decoder: RMSNorm, fused QKV projection, rotate-half RoPE,
causal grouped-query attention, output projection, RMSNorm, SwiGLU FFN, final RMSNorm and
an untied LM head.  No QK-norm, no biases.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It shares no code with the CUDA path and never imports it.

Pins (tests/test_oracle_pins.py): Eq. (1) closed form and the 262,144 B/token footnote,
RMSNorm/SwiGLU closed forms, RoPE invariants, brute-force loop attention on tiny inputs,
torch SDPA as a black-box library cross-check, causality between the full-sequence, the
chunk-by-chunk (cached-prefix) and the incremental code paths, the fp32 library matmul against
the fp64 one and against an error bound, the bf16 storage points against the library cast at
each of them, pack/unpack by a five-deep byte loop,
the whole forward (K, V and all logits) against the library's Llama decoder loaded with the same weights.
Every function of this module has a pin.  Outside what a pin can reach: agreement with the published
Qwen3/Llama checkpoints (no weights are available; the architecture is pinned, trained values are not involved).
"""
from __future__ import annotations

import numpy as np

# status codes of the assemble step; numerically equal to the C-ABI's codes by specification
OK = 0
ERR_ARG = -1
ERR_SHAPE = -2
ERR_BLOCK_RANGE = -3
ERR_BLOCK_ALIAS = -4
ERR_GAP = -5
ERR_OVERLAP = -6
ERR_SPLIT_UNALIGNED = -7
ERR_TABLE_SHORT = -8
ERR_WIRE_SIZE = -9
ERR_WORKSPACE = -10
ERR_STALE_EPOCH = -11
ERR_TOKEN_RANGE = -12


# --------------------------------------------------------------------------------------------
# Eq. (1): per-token KV footprint
# --------------------------------------------------------------------------------------------
def kv_bytes_per_token(n_layers: int, n_kv_heads: int, head_dim: int, elem_bytes: int = 2) -> int:
    """Eq. (1): s_KV = 2 * L * H_KV * d_h * b."""
    return 2 * n_layers * n_kv_heads * head_dim * elem_bytes


def kv_bytes(n_tokens: int, n_layers: int, n_kv_heads: int, head_dim: int, elem_bytes: int = 2) -> int:
    """Eq. (1): S_KV(N) = N * s_KV."""
    return n_tokens * kv_bytes_per_token(n_layers, n_kv_heads, head_dim, elem_bytes)


# --------------------------------------------------------------------------------------------
# bfloat16 image of the cache (the cache element type is 2 bytes, Section 1 footnote)
# --------------------------------------------------------------------------------------------
def to_bf16_bits(x) -> np.ndarray:
    """Round fp values to bfloat16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    return r.astype(np.uint16)


def from_bf16_bits(b) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------------------------
# Transformer pieces
# --------------------------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """h = x / sqrt(mean(x^2) + eps) * g, mean over the last (hidden) axis."""
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gain, dtype=np.float64)


def rope(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotate-half rotary embedding.  x: [T, H, d]; positions: [T] absolute 0-based positions.

    For j in [0, d/2): theta_j = base^(-2j/d), phi = pos * theta_j,
    (x_j, x_{j+d/2}) -> (x_j cos phi - x_{j+d/2} sin phi, x_{j+d/2} cos phi + x_j sin phi).
    """
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    half = d // 2
    j = np.arange(half, dtype=np.float64)
    theta = np.power(float(base), -2.0 * j / d)
    phi = np.asarray(positions, dtype=np.float64)[:, None] * theta[None, :]  # [T, d/2]
    c = np.cos(phi)[:, None, :]
    s = np.sin(phi)[:, None, :]
    a = x[..., :half]
    b = x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a, dtype=np.float64)
    return a / (1.0 + np.exp(-a))


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, q_pos0: int = 0) -> np.ndarray:
    """Causal grouped-query attention by explicit score matrices.

    q: [Tq, Hq, d] for absolute positions q_pos0 .. q_pos0+Tq-1; k, v: [Tk, Hkv, d] for
    positions 0 .. Tk-1.  Query head h reads KV head h // (Hq / Hkv).  Query i attends keys
    j <= q_pos0 + i.  Returns [Tq, Hq, d].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    tq, hq, d = q.shape
    tk, hkv, _ = k.shape
    group = hq // hkv
    scale = 1.0 / np.sqrt(d)
    qi = q_pos0 + np.arange(tq)[:, None]
    kj = np.arange(tk)[None, :]
    visible = kj <= qi
    out = np.empty_like(q)
    for h in range(hq):
        g = h // group
        s = (q[:, h, :] @ k[:, g, :].T) * scale
        s = np.where(visible, s, -np.inf)
        s = s - np.max(s, axis=1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=1, keepdims=True)
        out[:, h, :] = p @ v[:, g, :]
    return out


def _mm(x: np.ndarray, w: np.ndarray, mm_dtype) -> np.ndarray:
    """y = x @ w.T with W row-major [out, in]; library matmul in mm_dtype, result fp64."""
    if mm_dtype == np.float64:
        return np.asarray(x, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T
    return (np.asarray(x, dtype=mm_dtype) @ np.asarray(w, dtype=mm_dtype).T).astype(np.float64)


def _act(x: np.ndarray, act_bf16: bool) -> np.ndarray:
    """Optional bfloat16 storage point: the value as it exists after being stored in bf16."""
    return from_bf16_bits(to_bf16_bits(x)).astype(np.float64) if act_bf16 else x


def layer_forward(shape, w: dict, x: np.ndarray, positions: np.ndarray,
                  k_past=None, v_past=None, mm_dtype=np.float64, skip_after_kv: bool = False,
                  act_bf16: bool = False):
    """One decoder layer on rows x [T, D] at absolute `positions`.

    act_bf16 = False is the exact definition.  With act_bf16 every tensor that a 16-bit pipeline
    stores between contractions (normed activations, post-RoPE Q/K and V, attention output,
    SwiGLU output) is rounded to bfloat16 at that point while all arithmetic stays fp64: the
    same function evaluated at bf16 storage precision, which separates rounding that the
    2-byte cache/activation format makes unavoidable from arithmetic error.

    k_past/v_past: [P, Hkv, d] K/V of positions 0..P-1 already in the cache (None: P = 0);
    positions must equal P .. P+T-1.  Returns (x_out, k_new, v_new); k_new is post-RoPE.
    With skip_after_kv the layer stops once K/V exist (x_out is None): the last layer's K/V
    depend only on that layer's input.
    """
    t = x.shape[0]
    hq, hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    h = _act(rmsnorm(x, w["attn_norm"], shape.rms_eps), act_bf16)
    qkv = _mm(h, w["w_qkv"], mm_dtype)
    q = qkv[:, : hq * d].reshape(t, hq, d)
    k = qkv[:, hq * d: (hq + hkv) * d].reshape(t, hkv, d)
    v = _act(qkv[:, (hq + hkv) * d:].reshape(t, hkv, d), act_bf16)
    q = _act(rope(q, positions, shape.rope_base), act_bf16)
    k = _act(rope(k, positions, shape.rope_base), act_bf16)
    if skip_after_kv:
        return None, k, v
    if k_past is not None and len(k_past):
        k_all = np.concatenate([np.asarray(k_past, dtype=np.float64), k], axis=0)
        v_all = np.concatenate([np.asarray(v_past, dtype=np.float64), v], axis=0)
    else:
        k_all, v_all = k, v
    o = _act(attention(q, k_all, v_all, q_pos0=int(positions[0])), act_bf16)
    x = x + _mm(o.reshape(t, hq * d), w["w_o"], mm_dtype)
    h2 = _act(rmsnorm(x, w["ffn_norm"], shape.rms_eps), act_bf16)
    ab = _mm(h2, w["w_gate_up"], mm_dtype)
    m = _act(silu(ab[:, : shape.ffn]) * ab[:, shape.ffn:], act_bf16)
    x = x + _mm(m, w["w_down"], mm_dtype)
    return x, k, v


def forward_full(shape, head: dict, layers, token_ids, mm_dtype=np.float64,
                 want_logits: bool = True, all_logits: bool = False, act_bf16: bool = False):
    """Full-sequence forward over token_ids[0..T).

    `layers` is a callable l -> weight dict (so large models are generated layer by layer).
    Returns (K, V, logits): K, V fp64 [L, T, Hkv, d] (K post-RoPE); logits fp64 [V] for the
    last row ([T, V] with all_logits), or None when want_logits is False (the last layer then
    stops after its K/V).
    """
    token_ids = np.asarray(token_ids)
    t = len(token_ids)
    x = np.asarray(head["embed"], dtype=np.float64)[token_ids]
    pos = np.arange(t)
    ks, vs = [], []
    for l in range(shape.n_layers):
        last = (l == shape.n_layers - 1) and not want_logits
        x, k, v = layer_forward(shape, layers(l), x, pos, mm_dtype=mm_dtype, skip_after_kv=last,
                                act_bf16=act_bf16)
        ks.append(k)
        vs.append(v)
    logits = None
    if want_logits:
        rows = x if all_logits else x[-1:]
        logits = _mm(rmsnorm(rows, head["final_norm"], shape.rms_eps), head["lm_head"], mm_dtype)
        if not all_logits:
            logits = logits[0]
    return np.stack(ks), np.stack(vs), logits


def forward_chunked(shape, head: dict, layers, token_ids, chunk_sizes, mm_dtype=np.float64,
                    want_logits: bool = True, act_bf16: bool = False):
    """The same forward evaluated chunk by chunk (continued prefill, Section 4.5: the migration prefill is
    split into chunks that interleave with resident decoding).  Chunk c covers the next chunk_sizes[c] tokens;
    its rows attend to the K/V that earlier chunks left (k_past / v_past of `layer_forward`) and to
    themselves.  Returns (K, V, logits) like `forward_full`; logits are those of the last row of the last
    chunk.  `layers` is called once per (chunk, layer).
    """
    token_ids = np.asarray(token_ids)
    assert sum(chunk_sizes) == len(token_ids) and all(c > 0 for c in chunk_sizes)
    emb = np.asarray(head["embed"], dtype=np.float64)
    k_done = [np.zeros((0, shape.n_kv_heads, shape.head_dim)) for _ in range(shape.n_layers)]
    v_done = [np.zeros((0, shape.n_kv_heads, shape.head_dim)) for _ in range(shape.n_layers)]
    p0 = 0
    x = None
    for ci, c in enumerate(chunk_sizes):
        pos = np.arange(p0, p0 + c)
        x = emb[token_ids[p0:p0 + c]]
        final_chunk = ci == len(chunk_sizes) - 1
        for l in range(shape.n_layers):
            stop = final_chunk and (l == shape.n_layers - 1) and not want_logits
            x, k, v = layer_forward(shape, layers(l), x, pos, k_past=k_done[l], v_past=v_done[l],
                                    mm_dtype=mm_dtype, skip_after_kv=stop, act_bf16=act_bf16)
            k_done[l] = np.concatenate([k_done[l], k], axis=0)
            v_done[l] = np.concatenate([v_done[l], v], axis=0)
        p0 += c
    logits = None
    if want_logits:
        logits = _mm(rmsnorm(x[-1:], head["final_norm"], shape.rms_eps), head["lm_head"], mm_dtype)[0]
    return np.stack(k_done), np.stack(v_done), logits


def decode_step(shape, head: dict, layers, token_id: int, pos: int, k_cache, v_cache):
    """One incremental step for a single token at absolute position `pos`.

    k_cache, v_cache: [L, >=pos, Hkv, d] holding positions 0..pos-1.  Written as per-head
    vector arithmetic on one row (not through `attention`/`layer_forward`), so that equality
    with `forward_full` is a real check of causality rather than a tautology.
    Returns (k_new [L, Hkv, d], v_new [L, Hkv, d], logits [V]).
    """
    hq, hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    half = d // 2
    group = hq // hkv
    x = np.asarray(head["embed"], dtype=np.float64)[int(token_id)].copy()
    theta = np.array([float(shape.rope_base) ** (-2.0 * j / d) for j in range(half)])
    cs, sn = np.cos(pos * theta), np.sin(pos * theta)

    def rot(vec):
        a, b = vec[:half], vec[half:]
        return np.concatenate([a * cs - b * sn, b * cs + a * sn])

    k_new = np.empty((shape.n_layers, hkv, d))
    v_new = np.empty((shape.n_layers, hkv, d))
    for l in range(shape.n_layers):
        w = layers(l)
        h = x / np.sqrt(np.dot(x, x) / len(x) + shape.rms_eps) * np.asarray(w["attn_norm"], dtype=np.float64)
        qkv = np.asarray(w["w_qkv"], dtype=np.float64) @ h
        for g in range(hkv):
            k_new[l, g] = rot(qkv[(hq + g) * d: (hq + g + 1) * d])
            v_new[l, g] = qkv[(hq + hkv + g) * d: (hq + hkv + g + 1) * d]
        o = np.empty(hq * d)
        for hh in range(hq):
            g = hh // group
            qv = rot(qkv[hh * d: (hh + 1) * d])
            keys = np.concatenate([np.asarray(k_cache[l][:pos, g], dtype=np.float64), k_new[l, g][None]], axis=0)
            vals = np.concatenate([np.asarray(v_cache[l][:pos, g], dtype=np.float64), v_new[l, g][None]], axis=0)
            s = keys @ qv / np.sqrt(d)
            p = np.exp(s - s.max())
            p /= p.sum()
            o[hh * d: (hh + 1) * d] = p @ vals
        x = x + np.asarray(w["w_o"], dtype=np.float64) @ o
        h2 = x / np.sqrt(np.dot(x, x) / len(x) + shape.rms_eps) * np.asarray(w["ffn_norm"], dtype=np.float64)
        ab = np.asarray(w["w_gate_up"], dtype=np.float64) @ h2
        a, b = ab[: shape.ffn], ab[shape.ffn:]
        x = x + np.asarray(w["w_down"], dtype=np.float64) @ (a / (1.0 + np.exp(-a)) * b)
    hf = x / np.sqrt(np.dot(x, x) / len(x) + shape.rms_eps) * np.asarray(head["final_norm"], dtype=np.float64)
    logits = np.asarray(head["lm_head"], dtype=np.float64) @ hf
    return k_new, v_new, logits


# --------------------------------------------------------------------------------------------
# Paged cache: uint16 array [L, 2, num_blocks, Bs, Hkv, d]; page (l, kv, b) = cache[l, kv, b]
# --------------------------------------------------------------------------------------------
def new_cache(n_layers, num_blocks, block_size, n_kv_heads, head_dim, fill: int = 0) -> np.ndarray:
    return np.full((n_layers, 2, num_blocks, block_size, n_kv_heads, head_dim), fill, dtype=np.uint16)


def write_kv(cache: np.ndarray, k, v, block_table, pos0: int = 0) -> None:
    """Store K/V rows [L, T, Hkv, d] of positions pos0..pos0+T-1: page block_table[pos // Bs], slot pos % Bs."""
    bs = cache.shape[3]
    kb, vb = to_bf16_bits(k), to_bf16_bits(v)
    for i in range(kb.shape[1]):
        pos = pos0 + i
        blk = int(block_table[pos // bs])
        cache[:, 0, blk, pos % bs] = kb[:, i]
        cache[:, 1, blk, pos % bs] = vb[:, i]


def read_kv(cache: np.ndarray, block_table, n_tokens: int):
    """Logical K, V [L, n_tokens, Hkv, d] (fp32 values of the bf16 image) through a block table."""
    bs = cache.shape[3]
    nb = -(-n_tokens // bs)
    ids = np.asarray(block_table[:nb], dtype=np.int64)
    l, _, _, _, hkv, d = cache.shape
    k = cache[:, 0, ids].reshape(l, nb * bs, hkv, d)[:, :n_tokens]
    v = cache[:, 1, ids].reshape(l, nb * bs, hkv, d)[:, :n_tokens]
    return from_bf16_bits(k), from_bf16_bits(v)


def pack_blocks(cache: np.ndarray, block_ids) -> np.ndarray:
    """wire[i, l, kv] = page(l, kv, block_ids[i]) in logical order i (block-major wire), bytes verbatim."""
    l = cache.shape[0]
    page = cache.shape[3] * cache.shape[4] * cache.shape[5]
    wire = np.empty((len(block_ids), l, 2, page), dtype=np.uint16)
    for i, b in enumerate(block_ids):
        for layer in range(l):
            for kv in range(2):
                wire[i, layer, kv] = cache[layer, kv, int(b)].reshape(page)
    return wire


def check_assemble(num_blocks, block_size, logical, dst_ids, prefix_table, n_tokens_total,
                   epoch, expected_epoch) -> int:
    """State-consistency checks before activation (Section 4.3): returns a status code.

    The prefix must end on a block boundary (its table covers whole blocks); the suffix's
    logical blocks must be exactly {k/Bs .. ceil(n/Bs)-1}, each once ("without gaps or
    conflicts"); physical ids in range, pairwise distinct and disjoint from the prefix's;
    blocks of a cancelled attempt (stale epoch) never enter the active state.
    """
    if epoch != expected_epoch:
        return ERR_STALE_EPOCH
    n_prefix = len(prefix_table)
    n_suffix = len(dst_ids)
    if len(logical) != n_suffix or n_tokens_total < 0:
        return ERR_ARG
    total_blocks = -(-n_tokens_total // block_size)
    for b in list(prefix_table) + list(dst_ids):
        if not (0 <= int(b) < num_blocks):
            return ERR_BLOCK_RANGE
    phys = [int(b) for b in prefix_table] + [int(b) for b in dst_ids]
    if len(set(phys)) != len(phys):
        return ERR_BLOCK_ALIAS
    seen = set()
    for lb in logical:
        lb = int(lb)
        if lb < n_prefix or lb >= total_blocks or lb in seen:
            return ERR_OVERLAP
        seen.add(lb)
    if len(seen) != total_blocks - n_prefix:
        return ERR_GAP
    return OK


def unpack_assemble(cache: np.ndarray, wire: np.ndarray, logical, dst_ids, prefix_table,
                    n_tokens_total: int, epoch: int = 0, expected_epoch: int = 0):
    """page(l, kv, dst_ids[i]) = wire[i, l, kv]; merged table = prefix_table followed by the
    destination ids ordered by logical block.  On a failed check the cache is untouched.
    Returns (status, merged_table or None).
    """
    st = check_assemble(cache.shape[2], cache.shape[3], logical, dst_ids, prefix_table,
                        n_tokens_total, epoch, expected_epoch)
    if st != OK:
        return st, None
    l = cache.shape[0]
    if wire.shape[0] != len(dst_ids) or wire.shape[1] != l:
        return ERR_WIRE_SIZE, None
    n_prefix = len(prefix_table)
    merged = np.empty(n_prefix + len(dst_ids), dtype=np.int32)
    merged[:n_prefix] = prefix_table
    for i, b in enumerate(dst_ids):
        for layer in range(l):
            for kv in range(2):
                cache[layer, kv, int(b)] = wire[i, layer, kv].reshape(cache.shape[3:])
        merged[int(logical[i])] = int(b)
    return OK, merged
