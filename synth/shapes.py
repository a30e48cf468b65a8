"""Decoder shapes of the five benchmark configurations (random-init, no checkpoints)."""
from dataclasses import dataclass, asdict

MASTER_SEED = 260413519


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float
    rms_eps: float

    def n_params_matmul(self) -> int:
        """Parameters touched by one forward row (embedding table excluded)."""
        per_layer = self.d_model * self.head_dim * (2 * self.n_q_heads + 2 * self.n_kv_heads) \
            + 3 * self.d_model * self.d_ffn
        return self.n_layers * per_layer + self.vocab * self.d_model

    def asdict(self):
        return asdict(self)


SHAPES = {
    # tiny decoder: 2 layers, d=256, 4 heads of 64, FFN 1024, vocab 4096
    "tiny": ModelShape("tiny", 2, 256, 4, 4, 64, 1024, 4096, 10000.0, 1e-5),
    # Llama-3.2-1B-shaped
    "1b": ModelShape("1b", 16, 2048, 32, 8, 64, 8192, 128256, 500000.0, 1e-5),
    # Qwen3-8B-shaped
    "8b": ModelShape("8b", 36, 4096, 32, 8, 128, 12288, 151936, 1000000.0, 1e-6),
    # reduced-depth variants of the two large shapes: same per-layer tiles, fewer layers and a
    # smaller vocabulary, so that a CPU check of a whole forward finishes in seconds
    "1b-2l": ModelShape("1b-2l", 2, 2048, 32, 8, 64, 8192, 8192, 500000.0, 1e-5),
    "8b-2l": ModelShape("8b-2l", 2, 4096, 32, 8, 128, 12288, 8192, 1000000.0, 1e-6),
    # the 8B layer at four layers and a 32k vocabulary: a few GB on the device, for profiler captures
    "8b-4l": ModelShape("8b-4l", 4, 4096, 32, 8, 128, 12288, 32768, 1000000.0, 1e-6),
}
