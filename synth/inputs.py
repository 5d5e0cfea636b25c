"""Seeded generators: weights (rounded once to bfloat16), token ids, block ids, byte patterns."""
import numpy as np

from .configs import ModelShape

# request sizes (blocks) of the 16-request pack/unpack stress workload: drawn once from
# numpy.random.default_rng(0).integers(64, 513, 16) and recorded so nothing depends on the stream
STRESS_BLOCK_COUNTS = (445, 349, 293, 185, 202, 82, 97, 71, 142, 429, 355, 473, 290, 336, 499, 391)

# multiplier of the counter-based 64-bit fill pattern (splitmix64 constants)
PATTERN_MUL = (0x9E3779B97F4A7C15, 0xBF58476D1CE4E5B9, 0x94D049BB133111EB)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even; NaN stays NaN."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    out = np.where(nan, (u >> np.uint32(16)) | np.uint32(0x40), rounded)
    return out.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round_f32(x: np.ndarray) -> np.ndarray:
    """Values of x rounded to bfloat16, returned as float32 (exactly representable)."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(s) for s in stream]])


def _matrix(shape: ModelShape, rng, out_dim: int, in_dim: int) -> np.ndarray:
    std = (1.0 / np.sqrt(in_dim)) if shape.sharp else shape.init_std
    w = rng.standard_normal((out_dim, in_dim), dtype=np.float32) * np.float32(std)
    return bf16_round_f32(w)


def _gain(shape: ModelShape, rng, dim: int) -> np.ndarray:
    if shape.sharp:
        return bf16_round_f32(rng.uniform(0.5, 1.5, dim).astype(np.float32))
    return np.ones(dim, dtype=np.float32)


def layer_weights(shape: ModelShape, seed: int, layer: int) -> dict:
    """Weights of one decoder layer, float32 arrays holding bfloat16-representable values.

    Row-major [out, in]: w_qkv rows ordered Q | K | V (heads contiguous), w_gate_up rows gate | up.
    """
    rng = _rng(seed, 1, layer)
    return {
        "attn_norm": _gain(shape, rng, shape.hidden),
        "w_qkv": _matrix(shape, rng, shape.qkv_dim, shape.hidden),
        "w_o": _matrix(shape, rng, shape.hidden, shape.q_dim),
        "ffn_norm": _gain(shape, rng, shape.hidden),
        "w_gate_up": _matrix(shape, rng, 2 * shape.ffn, shape.hidden),
        "w_down": _matrix(shape, rng, shape.hidden, shape.ffn),
    }


def head_weights(shape: ModelShape, seed: int) -> dict:
    """Embedding table, final norm gain and (untied) LM head."""
    rng = _rng(seed, 2)
    return {
        "embed": _matrix(shape, rng, shape.vocab, shape.hidden) if not shape.sharp else
        bf16_round_f32(rng.standard_normal((shape.vocab, shape.hidden), dtype=np.float32)),
        "final_norm": _gain(shape, rng, shape.hidden),
        "lm_head": _matrix(shape, rng, shape.vocab, shape.hidden),
    }


def token_ids(shape: ModelShape, seed: int, n: int) -> np.ndarray:
    """n token ids uniform in [0, vocab), int32."""
    return _rng(seed, 3).integers(0, shape.vocab, n).astype(np.int32)


def block_permutation(seed: int, num_blocks: int) -> np.ndarray:
    """A seeded permutation of physical block ids: fragmented, non-monotone tables are slices of it."""
    return _rng(seed, 4).permutation(num_blocks).astype(np.int32)


def pattern_bytes(seed: int, byte_offset: int, n_bytes: int) -> np.ndarray:
    """Counter-based fill pattern: the 64-bit word at index w (byte offset 8w) is splitmix64(seed, w).

    byte_offset and n_bytes must be multiples of 8.  Returns uint8[n_bytes] (little endian words).
    A device fill kernel implementing the same counter function reproduces any page on its own.
    """
    assert byte_offset % 8 == 0 and n_bytes % 8 == 0
    w = np.arange(byte_offset // 8, (byte_offset + n_bytes) // 8, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (w + np.uint64(seed)) * np.uint64(PATTERN_MUL[0])
        z = (z ^ (z >> np.uint64(30))) * np.uint64(PATTERN_MUL[1])
        z = (z ^ (z >> np.uint64(27))) * np.uint64(PATTERN_MUL[2])
        z = z ^ (z >> np.uint64(31))
    return z.view(np.uint8)
