"""Seeded random-init weights: N(0, 0.02^2) rounded to bf16, norm gains equal to one.

Counter-based: every tensor (and every 4 Mi-element block of it) has its own Philox key, so a
tensor's values do not depend on which other tensors were generated or in what order, and blocks
can be produced by several threads.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

from .shapes import ModelShape, MASTER_SEED

_BLOCK = 1 << 22
_STD = 0.02


def tensor_names(shape: ModelShape):
    """(name, (rows, cols)) of every matrix, in blob order.  All are [out_features][in_features]."""
    s = shape
    out = [("embed", (s.vocab, s.d_model))]
    for l in range(s.n_layers):
        out += [
            (f"l{l}.wq", (s.n_q_heads * s.head_dim, s.d_model)),
            (f"l{l}.wk", (s.n_kv_heads * s.head_dim, s.d_model)),
            (f"l{l}.wv", (s.n_kv_heads * s.head_dim, s.d_model)),
            (f"l{l}.wo", (s.d_model, s.n_q_heads * s.head_dim)),
            (f"l{l}.wg", (s.d_ffn, s.d_model)),
            (f"l{l}.wu", (s.d_ffn, s.d_model)),
            (f"l{l}.wd", (s.d_model, s.d_ffn)),
        ]
    out.append(("lm_head", (s.vocab, s.d_model)))
    return out


def _fill_block(dst: np.ndarray, seed: int, tid: int, blk: int):
    g = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ tid, blk]))
    dst[:] = g.standard_normal(dst.shape[0], dtype=np.float32)


def _gaussian_bf16(seed: int, tid: int, rows: int, cols: int, pool) -> torch.Tensor:
    n = rows * cols
    buf = np.empty(n, dtype=np.float32)
    nblk = (n + _BLOCK - 1) // _BLOCK
    futs = [pool.submit(_fill_block, buf[b * _BLOCK:min(n, (b + 1) * _BLOCK)], seed, tid, b)
            for b in range(nblk)]
    for f in futs:
        f.result()
    t = torch.from_numpy(buf).mul_(_STD).to(torch.bfloat16)   # round-to-nearest-even
    return t.view(rows, cols)


def _gain(shape: ModelShape, gain_seed, which: int) -> torch.Tensor:
    """Norm gain vector: ones (the benchmark configurations), or, with a gain seed, 1 + 0.3 N(0,1) so that a test
    can tell the gain vectors of different layers and norms apart."""
    if gain_seed is None:
        return torch.ones(shape.d_model, dtype=torch.float32)
    g = np.random.Generator(np.random.Philox(key=[(int(gain_seed) << 20) ^ 0x6A17, which]))
    return torch.from_numpy(1.0 + 0.3 * g.standard_normal(shape.d_model)).to(torch.float32)


def make_weights(shape: ModelShape, seed: int = MASTER_SEED, layers=None, with_globals: bool = True,
                 gain_seed=None):
    """dict name -> torch.bfloat16 CPU tensor [out][in]; norm gains (fp32; all ones unless `gain_seed`
    is given, then 1 + 0.3 N(0,1) per element) under 'l{l}.g1', 'l{l}.g2', 'gf'.  `layers` restricts
    generation to some layer indices; the global tensors (embedding, LM head, final gain) are produced
    unless `with_globals` is false.  A tensor's values depend only on (seed, its index in tensor_names),
    so a model can be generated piece by piece."""
    w = {}
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as pool:
        for tid, (name, (r, c)) in enumerate(tensor_names(shape)):
            per_layer = name.startswith("l") and name[1].isdigit()
            if per_layer and layers is not None and int(name[1:name.index(".")]) not in layers:
                continue
            if not per_layer and not with_globals:
                continue
            w[name] = _gaussian_bf16(seed, tid, r, c, pool)
    for l in range(shape.n_layers):
        if layers is not None and l not in layers:
            continue
        w[f"l{l}.g1"] = _gain(shape, gain_seed, 2 * l)
        w[f"l{l}.g2"] = _gain(shape, gain_seed, 2 * l + 1)
    w["gf"] = _gain(shape, gain_seed, 2 * shape.n_layers)
    return w
