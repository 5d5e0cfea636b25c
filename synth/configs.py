"""Model and cache shapes of the synthetic workloads (decoder-only GQA transformer shapes)."""
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_base: float = 1.0e6
    rms_eps: float = 1.0e-6
    block_size: int = 16
    init_std: float = 0.02
    sharp: bool = False  # "sharp" init: std 1/sqrt(fan_in), norm gains U(0.5, 1.5)

    def with_layers(self, n_layers: int) -> "ModelShape":
        return replace(self, n_layers=n_layers, name=f"{self.name}-L{n_layers}")

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def qkv_dim(self) -> int:
        return self.q_dim + 2 * self.kv_dim


def kv_page_bytes(shape: ModelShape, elem_bytes: int = 2) -> int:
    """Bytes of one page: one layer, K or V, one block of `block_size` tokens."""
    return shape.block_size * shape.n_kv_heads * shape.head_dim * elem_bytes


SHAPES = {
    # tiny decoder used for full-depth parity (prefix 128 + suffix 32, block size 16)
    "tiny": ModelShape("tiny", n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64,
                       ffn=512, vocab=1024),
    "tiny-sharp": ModelShape("tiny-sharp", n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2,
                             head_dim=64, ffn=512, vocab=1024, sharp=True),
    # Qwen3-8B-shaped (shapes only: no QK-norm, no biases, untied embeddings)
    "8b": ModelShape("8b", n_layers=36, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128,
                     ffn=12288, vocab=151936),
    # Qwen3-32B-shaped: 256 KiB of KV per token
    "32b": ModelShape("32b", n_layers=64, hidden=5120, n_q_heads=64, n_kv_heads=8, head_dim=128,
                      ffn=25600, vocab=151936),
}
