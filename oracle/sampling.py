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


def accept_sampled_tree(logits: torch.Tensor, z: Sequence[int], parents: Sequence[int], temperature: float,
                        u: Sequence[float]):
    """Speculative sampling over a draft tree (Appendix A.1's tree + Appendix B.2's acceptance rule).  z: tokens of
    all k nodes (z[0] = pending), parents[0] = -1.  At node v with target p = softmax(logits_v / T) the children are
    tried in node order against the residual: child c (token x) is accepted with probability r(x) / R, where r is
    p with the tokens of the children already refused removed and R its total; u[c] decides child c.  If a child
    is accepted the walk moves there; if none is (or v is a leaf) one sample of the residual is emitted with u[0]
    and the step ends.  Each emitted token is then distributed as the model's own, whatever the tree holds.
    Returns (path of node indices, emitted ids)."""
    k = len(z)
    assert logits.shape[0] == k and len(parents) == k and len(u) == k
    path, emitted, v = [0], [], 0
    while True:
        r = target_probs(logits[v], temperature).clone()
        nxt = None
        for c in range(v + 1, k):
            if parents[c] != v:
                continue
            x = z[c]
            if u[c] * float(r.sum()) < float(r[x]):
                nxt = c
                break
            r[x] = 0.0
        if nxt is None:
            emitted.append(sample_inverse_cdf(r, u[0]))
            return path, emitted
        path.append(nxt)
        emitted.append(z[nxt])
        v = nxt
