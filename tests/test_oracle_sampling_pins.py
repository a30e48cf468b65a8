"""Pins for the speculative-sampling oracle (Appendix B.2: speculative sampling as the acceptance
strategy): the distribution of what is emitted must be the model's own, whatever the drafts are; the
limit T -> 0 is greedy acceptance; the inverse-CDF draw against a brute-force loop."""
import math

import numpy as np
import torch

import oracle
from oracle.transformer import F64


def test_inverse_cdf_equals_a_plain_loop():
    g = np.random.Generator(np.random.Philox(key=[11, 1]))
    for _ in range(200):
        n = int(g.integers(1, 40))
        w = torch.tensor(g.random(n) * (g.random(n) > 0.3), dtype=F64)
        if float(w.sum()) == 0.0:
            w[int(g.integers(0, n))] = 1.0
        u = float(g.random())
        acc, want = 0.0, None
        target = u * float(w.sum())
        for i in range(n):
            acc += float(w[i])
            if acc > target:
                want = i
                break
        if want is None:
            want = n - 1
        assert oracle.sample_inverse_cdf(w, u) == want
        assert float(w[oracle.sample_inverse_cdf(w, u)]) > 0.0 or want == n - 1
    assert oracle.sample_inverse_cdf(torch.tensor([0.0, 2.0, 0.0, 1.0], dtype=F64), 0.0) == 1
    assert oracle.sample_inverse_cdf(torch.tensor([0.0, 2.0, 0.0, 1.0], dtype=F64), 0.7) == 3


def test_target_probs_is_softmax_over_temperature():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(50, generator=g, dtype=F64) * 3
    for T in (0.3, 1.0, 2.5):
        assert torch.allclose(oracle.target_probs(x, T), torch.softmax(x / T, dim=0), rtol=0, atol=1e-15)


def test_low_temperature_is_greedy_acceptance():
    g = np.random.Generator(np.random.Philox(key=[11, 2]))
    for _ in range(50):
        k, V = int(g.integers(1, 7)), 30
        logits = torch.tensor(g.normal(size=(k, V)) * 4, dtype=F64)
        t = oracle.argmax_lowest(logits)
        draft = [t[j] if g.random() < 0.7 else int(g.integers(0, V)) for j in range(k - 1)]
        l_ref = 0
        while l_ref < k - 1 and t[l_ref] == draft[l_ref]:
            l_ref += 1
        u = [float(x) for x in g.random(k) * 0.98 + 0.01]
        l, em = oracle.accept_sampled(logits, draft, 1e-4, u)
        assert l == l_ref and em == draft[:l_ref] + [t[l_ref]]


def _chi2(counts, probs):
    n = counts.sum()
    keep = probs * n >= 5
    return float((((counts - probs * n) ** 2) / (probs * n))[keep].sum()), int(keep.sum()) - 1


def test_emitted_tokens_follow_the_model_distribution_whatever_the_draft():
    """The theorem behind speculative sampling: the first emitted token ~ p_0 and, given that the
    first draft was accepted, the second ~ p_1 -- for a likely, an unlikely and a random draft."""
    g = np.random.Generator(np.random.Philox(key=[11, 3]))
    V, T, n = 12, 0.8, 40000
    logits = torch.tensor(g.normal(size=(3, V)) * 1.5, dtype=F64)
    p0 = oracle.target_probs(logits[0], T).numpy()
    p1 = oracle.target_probs(logits[1], T).numpy()
    for d0 in (int(np.argmax(p0)), int(np.argmin(p0)), 5):
        draft = [d0, int(np.argmax(p1))]
        first = np.zeros(V)
        second = np.zeros(V)
        acc0 = 0
        us = g.random((n, 3))
        for i in range(n):
            l, em = oracle.accept_sampled(logits, draft, T, [float(x) for x in us[i]])
            first[em[0]] += 1
            if l >= 1:
                acc0 += 1
                second[em[1]] += 1
        c, dof = _chi2(first, p0)
        assert c < dof + 5 * math.sqrt(2 * dof), (d0, c, dof)          # about 5 sigma of a chi-square
        if acc0 >= 1000:                                               # enough accepted first drafts to test row 1
            c, dof = _chi2(second, p1)
            assert dof >= 3 and c < dof + 5 * math.sqrt(2 * dof), (d0, c, dof)
        assert abs(acc0 / n - p0[d0]) < 5 * math.sqrt(p0[d0] * (1 - p0[d0]) / n) + 1e-9   # P(accept) = p(x)


def test_tree_rule_on_a_chain_is_the_chain_rule():
    """With parents j - 1 the tree walk is the chain rule, the uniforms renamed: node c's uniform is the chain's
    u[c - 1], the tree's u[0] is the chain's sample uniform u[k - 1]."""
    g = np.random.Generator(np.random.Philox(key=[11, 4]))
    for _ in range(100):
        k, V = int(g.integers(1, 7)), 20
        logits = torch.tensor(g.normal(size=(k, V)) * 2, dtype=F64)
        draft = [int(x) for x in g.integers(0, V, size=k - 1)]
        T = float(g.choice([0.3, 1.0]))
        u = [float(x) for x in g.random(k)]
        l, em = oracle.accept_sampled(logits, draft, T, u)
        ut = [u[k - 1]] + u[:k - 1]
        path, em_t = oracle.accept_sampled_tree(logits, [7] + draft, [-1] + list(range(k - 1)), T, ut)
        assert path == list(range(l + 1)) and em_t == em


def test_tree_sampling_emits_the_model_distribution():
    """Several candidates at the root and below its first child: the first emitted token follows p_0 and, given
    that the walk took child 1, the second follows p_1 -- the residual bookkeeping is what makes this true."""
    g = np.random.Generator(np.random.Philox(key=[11, 5]))
    V, T, n = 10, 0.9, 40000
    z = [0, 3, 7, 1, 4, 5]            # root; children of the root: 3, 7, 1 (nodes 1..3); children of node 1: 4, 5
    parents = [-1, 0, 0, 0, 1, 1]
    logits = torch.tensor(g.normal(size=(6, V)) * 1.2, dtype=F64)
    p0 = oracle.target_probs(logits[0], T).numpy()
    p1 = oracle.target_probs(logits[1], T).numpy()
    order = [int(i) for i in np.argsort(-p0)]
    z[1], z[2], z[3] = order[0], order[5], order[2]       # a likely first child, then an unlikely and a likely one
    first, second, took1 = np.zeros(V), np.zeros(V), 0
    us = g.random((n, 6))
    for i in range(n):
        path, em = oracle.accept_sampled_tree(logits, z, parents, T, [float(x) for x in us[i]])
        first[em[0]] += 1
        if len(path) > 1 and path[1] == 1:
            took1 += 1
            second[em[1]] += 1
    c, dof = _chi2(first, p0)
    assert c < dof + 5 * math.sqrt(2 * dof), (c, dof)
    c, dof = _chi2(second, p1)
    assert took1 > 2000 and c < dof + 5 * math.sqrt(2 * dof), (c, dof)
    assert abs(took1 / n - p0[z[1]]) < 5 * math.sqrt(p0[z[1]] * (1 - p0[z[1]]) / n)   # the first child is taken with p(x)
