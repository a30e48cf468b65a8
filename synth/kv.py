"""Seeded synthetic KV cache contents for long contexts (values exactly representable in bf16)."""
import numpy as np
import torch

from .shapes import ModelShape, MASTER_SEED


def make_synthetic_kv(shape: ModelShape, length: int, seed: int = MASTER_SEED, stream: int = 0,
                      layers=None):
    """Returns (K, V): lists over layers of torch.bfloat16 [length][n_kv_heads][head_dim],
    entries ~ N(0,1) rounded to bf16."""
    K, V = [], []
    for l in (range(shape.n_layers) if layers is None else layers):
        g = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ (0xABC00 + stream), l]))
        n = length * shape.n_kv_heads * shape.head_dim
        k = torch.from_numpy(g.standard_normal(n, dtype=np.float32)).to(torch.bfloat16)
        v = torch.from_numpy(g.standard_normal(n, dtype=np.float32)).to(torch.bfloat16)
        K.append(k.view(length, shape.n_kv_heads, shape.head_dim))
        V.append(v.view(length, shape.n_kv_heads, shape.head_dim))
    return K, V
