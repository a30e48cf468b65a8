"""CPU oracle for the verification forward: a plain decoder-only transformer in float64.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this module; it exists so that
tests, the smoke check and the benchmark's cpu_baseline leg have an independent, slow, obviously
correct statement of what the verify step computes.  It shares no code with the CUDA path.

What is computed (paper: Section 4.1 "verifies these draft candidates in parallel and accepts the
longest prefix"; Appendix A.1 "single forward pass" over the flattened drafts; Algorithm 1,
steps Verification / SelectLongestAcceptedPrefix / append):

  * forward of a pre-norm decoder (RMSNorm, rotary embedding in the rotate-half pairing,
    grouped-query attention, SwiGLU MLP, untied LM head) — the layer recipe is fixed by the
    benchmark configurations, the paper only says "target model";
  * two drivers over the same row arithmetic: full recompute of a whole sequence, and an
    incremental chunk forward against cached K/V (contiguous arrays, no paging);
  * vanilla greedy decoding (argmax, lowest id on ties);
  * one speculative step: chunk = pending token + drafts, accepted length = longest draft prefix
    that equals the per-position argmax, plus the bonus token.

Arithmetic: weights are bf16-rounded values (given), widened exactly to float64; every
intermediate is float64.  Parity status of the pieces is listed in tests/test_oracle_pins.py;
absolute logit values are pinned only through invariants (no trained weights exist here).
"""
import math
from typing import List, Optional, Sequence

import torch

F64 = torch.float64


def _wt(x: torch.Tensor, w: torch.Tensor, chunk_rows: int = 1 << 14) -> torch.Tensor:
    """x[T, in] @ w[out, in]^T with w widened to float64 a block of rows at a time."""
    outs = []
    for r0 in range(0, w.shape[0], chunk_rows):
        outs.append(x @ w[r0:r0 + chunk_rows].to(F64).T)
    return outs[0] if len(outs) == 1 else torch.cat(outs, dim=1)


def rmsnorm(x: torch.Tensor, g: torch.Tensor, eps: float) -> torch.Tensor:
    """x * rsqrt(mean(x^2) + eps) * g, row-wise."""
    ms = (x * x).mean(dim=-1, keepdim=True)
    return x / torch.sqrt(ms + eps) * g.to(F64)


def rope(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding, rotate-half pairing: element i is paired with i + hd/2 and the pair is
    rotated by the angle pos * theta^(-2i/hd).  x: [T, H, hd], pos: [T] integer positions."""
    hd = x.shape[-1]
    half = hd // 2
    i = torch.arange(half, dtype=F64)
    inv_freq = theta ** (-2.0 * i / hd)
    ang = pos.to(F64)[:, None] * inv_freq[None, :]          # [T, half]
    c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * c - x2 * s, x2 * c + x1 * s], dim=-1)


def attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, q_pos: torch.Tensor,
              k_pos: torch.Tensor, allowed: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Grouped-query attention.  q: [Tq, Hq, hd]; k, v: [Tk, Hkv, hd].  By default causal: a query
    at position p attends to every key at position <= p.  `allowed` ([Tq, Tk] bool) replaces that
    rule (the tree-structured mask of Appendix A.1).  Query head h uses kv head h // (Hq / Hkv).
    Returns [Tq, Hq, hd]."""
    Tq, Hq, hd = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(hd)
    if allowed is None:
        allowed = k_pos[None, :] <= q_pos[:, None]          # [Tq, Tk]
    out = torch.empty_like(q)
    for h in range(Hq):
        kh = h // G
        s = (q[:, h, :] @ k[:, kh, :].T) * scale            # [Tq, Tk]
        s = s.masked_fill(~allowed, float("-inf"))
        s = s - s.max(dim=-1, keepdim=True).values
        p = torch.exp(s)
        p = p / p.sum(dim=-1, keepdim=True)
        out[:, h, :] = p @ v[:, kh, :]
    return out


def swiglu(gate: torch.Tensor, up: torch.Tensor) -> torch.Tensor:
    """silu(gate) * up with silu(x) = x / (1 + exp(-x))."""
    return gate / (1.0 + torch.exp(-gate)) * up


def argmax_lowest(logits: torch.Tensor) -> List[int]:
    """Per-row argmax; among equal maxima the lowest token id."""
    out = []
    for row in logits:
        m = row.max()
        out.append(int(torch.nonzero(row == m)[0, 0]))
    return out


class KVCache:
    """Contiguous per-layer K/V of one sequence: lists of float64 [len, Hkv, hd]."""

    def __init__(self, n_layers: int, n_kv_heads: int, head_dim: int):
        self.k = [torch.zeros(0, n_kv_heads, head_dim, dtype=F64) for _ in range(n_layers)]
        self.v = [torch.zeros(0, n_kv_heads, head_dim, dtype=F64) for _ in range(n_layers)]

    @property
    def length(self) -> int:
        return self.k[0].shape[0]

    def truncate(self, n: int):
        self.k = [t[:n] for t in self.k]
        self.v = [t[:n] for t in self.v]

    def import_kv(self, K: Sequence[torch.Tensor], V: Sequence[torch.Tensor]):
        self.k = [t.to(F64) for t in K]
        self.v = [t.to(F64) for t in V]

    def clone(self) -> "KVCache":
        c = KVCache.__new__(KVCache)
        c.k = [t.clone() for t in self.k]
        c.v = [t.clone() for t in self.v]
        return c


class OracleModel:
    def __init__(self, shape, weights: dict):
        """shape: object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab,
        rope_theta, rms_eps.  weights: name -> tensor ([out][in] matrices, gain vectors)."""
        self.s = shape
        self.w = weights

    def new_cache(self) -> KVCache:
        return KVCache(self.s.n_layers, self.s.n_kv_heads, self.s.head_dim)

    # -- the row arithmetic shared by both drivers ------------------------------------------
    def _layer(self, l: int, x: torch.Tensor, pos: torch.Tensor, k_prev, v_prev, pos_prev,
               probe: Optional[dict] = None, allowed: Optional[torch.Tensor] = None):
        xs, k_alls, v_alls = self._layer_multi(l, [x], [pos], [k_prev], [v_prev], [pos_prev], probe,
                                               None if allowed is None else [allowed])
        return xs[0], k_alls[0], v_alls[0]

    def _layer_multi(self, l: int, xs, poss, k_prevs, v_prevs, pos_prevs, probe: Optional[dict] = None,
                     alloweds=None):
        """One decoder layer over several independent sequences (a batched step): sequence i has rows
        xs[i] at positions poss[i] behind its own cached k_prevs[i], v_prevs[i].  Norms, projections
        and the MLP act on rows, so they run once over all rows; attention runs per sequence.
        Returns (new rows, all keys, all values), each a list over the sequences."""
        s, w = self.s, self.w
        n_rows = [x.shape[0] for x in xs]
        x = torch.cat(list(xs), dim=0)
        pos = torch.cat(list(poss))
        T = x.shape[0]
        h = rmsnorm(x, w[f"l{l}.g1"], s.rms_eps)
        q = _wt(h, w[f"l{l}.wq"]).view(T, s.n_q_heads, s.head_dim)
        k = _wt(h, w[f"l{l}.wk"]).view(T, s.n_kv_heads, s.head_dim)
        v = _wt(h, w[f"l{l}.wv"]).view(T, s.n_kv_heads, s.head_dim)
        q = rope(q, pos, s.rope_theta)
        k = rope(k, pos, s.rope_theta)
        o_parts, k_alls, v_alls = [], [], []
        r0 = 0
        for i, n in enumerate(n_rows):
            k_all = torch.cat([k_prevs[i], k[r0:r0 + n]], dim=0)
            v_all = torch.cat([v_prevs[i], v[r0:r0 + n]], dim=0)
            pos_all = torch.cat([pos_prevs[i], poss[i]])
            o_parts.append(attention(q[r0:r0 + n], k_all, v_all, poss[i], pos_all,
                                     None if alloweds is None else alloweds[i]))
            k_alls.append(k_all)
            v_alls.append(v_all)
            r0 += n
        o = torch.cat(o_parts, dim=0).reshape(T, s.n_q_heads * s.head_dim)
        x = x + _wt(o, w[f"l{l}.wo"])
        h2 = rmsnorm(x, w[f"l{l}.g2"], s.rms_eps)
        a = swiglu(_wt(h2, w[f"l{l}.wg"]), _wt(h2, w[f"l{l}.wu"]))
        x = x + _wt(a, w[f"l{l}.wd"])
        if probe is not None:
            probe[f"l{l}.q"], probe[f"l{l}.k"], probe[f"l{l}.v"] = q, k, v
            probe[f"l{l}.attn"], probe[f"l{l}.act"], probe[f"l{l}.x"] = o, a, x
        return list(torch.split(x, n_rows, dim=0)), k_alls, v_alls

    def _head(self, x: torch.Tensor) -> torch.Tensor:
        return _wt(rmsnorm(x, self.w["gf"], self.s.rms_eps), self.w["lm_head"])

    # -- driver 1: full recompute -------------------------------------------------------------
    def forward_full(self, tokens: Sequence[int], pos_offset: int = 0,
                     probe: Optional[dict] = None) -> torch.Tensor:
        """Logits [T, V] for every position of `tokens`, everything recomputed from scratch."""
        s = self.s
        T = len(tokens)
        pos = torch.arange(T) + pos_offset
        x = self.w["embed"][torch.tensor(list(tokens))].to(F64)
        e = torch.zeros(0, s.n_kv_heads, s.head_dim, dtype=F64)
        for l in range(s.n_layers):
            x, _, _ = self._layer(l, x, pos, e, e, pos[:0], probe)
        return self._head(x)

    # -- driver 2: incremental chunk against a cache ------------------------------------------
    def forward_chunk(self, tokens: Sequence[int], cache: KVCache,
                      probe: Optional[dict] = None) -> torch.Tensor:
        """Logits [k, V] for a chunk placed at positions [len, len+k) after the cached prefix.
        The chunk's K/V are appended to the cache (the caller truncates on rejection)."""
        s = self.s
        n0, k = cache.length, len(tokens)
        pos = torch.arange(k) + n0
        pos_prev = torch.arange(n0)
        x = self.w["embed"][torch.tensor(list(tokens))].to(F64)
        for l in range(s.n_layers):
            x, cache.k[l], cache.v[l] = self._layer(l, x, pos, cache.k[l], cache.v[l], pos_prev,
                                                    probe)
        if probe is not None:
            probe["x_final"] = x
        return self._head(x)

    # -- vanilla greedy -----------------------------------------------------------------------
    def greedy_next(self, pending: int, cache: KVCache) -> int:
        return argmax_lowest(self.forward_chunk([pending], cache))[0]

    # -- one speculative step -----------------------------------------------------------------
    def verify(self, pending: int, draft: Sequence[int], cache: KVCache, want_logits=False):
        """Chunk z = [pending, d_1..d_g].  t_j = argmax of row j.  l = largest n with
        t_j == d_{j+1} for all j < n.  Emits d_1..d_l followed by t_l; the cache keeps
        pending and the l accepted drafts (length += l + 1).
        Returns dict(accept_len, emitted, argmax[, logits])."""
        z = [pending] + list(draft)
        n0 = cache.length
        logits = self.forward_chunk(z, cache)
        t = argmax_lowest(logits)
        l = 0
        while l < len(draft) and t[l] == draft[l]:
            l += 1
        cache.truncate(n0 + l + 1)
        res = dict(accept_len=l, emitted=list(draft[:l]) + [t[l]], argmax=t)
        if want_logits:
            res["logits"] = logits
        return res


def topk_lowest(logits_row: torch.Tensor, k: int) -> List[int]:
    """The k ids with the highest logits, best first, lowest id on ties."""
    v = logits_row.tolist()
    return sorted(range(len(v)), key=lambda i: (-v[i], i))[:k]


def top2_gap(logits_row: torch.Tensor) -> float:
    """Difference between the largest and second-largest logit of a row."""
    v = torch.topk(logits_row, 2).values
    return float(v[0] - v[1])
