"""CPU oracle for speculative-sampling acceptance at temperature T > 0.

TEST INFRASTRUCTURE ONLY (see oracle/transformer.py).

Paper: Appendix B.2 adopts speculative sampling as the acceptance strategy (Section 5.1 names it
too).  The drafts here come from retrieval or the schema, so the draft distribution q is a point
mass on the drafted token x, and the rule of speculative sampling becomes: with the target
distribution p = softmax(logits / T) of the row that predicts x,

    accept x                      with probability min(1, p(x) / q(x)) = p(x);
    otherwise emit one sample of  norm(max(p - q, 0)) = p with x removed, renormalised, and stop;
    if every draft was accepted   emit one sample of the last row's p (the bonus token).

The emitted stream is then distributed exactly as sampling from the model token by token, whatever
the drafts are.  All random numbers are inputs: u[j] in [0, 1) decides draft j + 1 (j < k - 1), and
u[k - 1] draws the one sample of the step.  A sample is taken by inverse CDF in index order: the
smallest i with w_0 + ... + w_i > u * (w_0 + ... + w_{V-1}).
"""
from typing import Sequence

import torch

from .transformer import OracleModel, KVCache, F64


def target_probs(logits_row: torch.Tensor, temperature: float) -> torch.Tensor:
    z = logits_row.to(F64) / temperature
    z = z - z.max()
    w = torch.exp(z)
    return w / w.sum()


def sample_inverse_cdf(w: torch.Tensor, u: float) -> int:
    """Smallest index whose running sum exceeds u * total (weights >= 0, not all zero)."""
    c = torch.cumsum(w.to(F64), dim=0)
    i = int(torch.searchsorted(c, torch.tensor(u * float(c[-1]), dtype=F64), right=True))
    return min(i, w.numel() - 1)


def accept_sampled(logits: torch.Tensor, draft: Sequence[int], temperature: float, u: Sequence[float]):
    """logits: [k, V] of the chunk [pending, draft...]; u: k uniforms.  Returns (accept_len, emitted)."""
    k = logits.shape[0]
    assert k == len(draft) + 1 and len(u) == k
    for j, x in enumerate(draft):
        p = target_probs(logits[j], temperature)
        if u[j] < float(p[x]):
            continue
        p = p.clone()
        p[x] = 0.0
        return j, list(draft[:j]) + [sample_inverse_cdf(p, u[k - 1])]
    p = target_probs(logits[k - 1], temperature)
    return k - 1, list(draft) + [sample_inverse_cdf(p, u[k - 1])]


def verify_sampled(model: OracleModel, pending: int, draft: Sequence[int], cache: KVCache,
                   temperature: float, u: Sequence[float], want_logits: bool = False):
    """One speculative step with sampling acceptance; the cache keeps pending + the accepted drafts."""
    z = [pending] + list(draft)
    n0 = cache.length
    logits = model.forward_chunk(z, cache)
    l, emitted = accept_sampled(logits, draft, temperature, u)
    cache.truncate(n0 + l + 1)
    res = dict(accept_len=l, emitted=emitted)
    if want_logits:
        res["logits"] = logits
    return res
