"""ts_verify_sampled against the oracle's speculative-sampling acceptance (Appendix B.2), with the same
uniforms on both sides: accepted length and emitted ids, trial after trial on one staged context.  A decision
taken on floating point may differ only where the oracle's own margin is within the logit tolerance: an accept
test with |u - p(x)| small, or a sample whose uniform lies next to the boundary of the GPU's id in the
oracle's CDF."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from gpu_util import make_pair, synthetic_context, LOGIT_MAX_ABS

pytestmark = pytest.mark.gpu


def _near_boundary(logits_row, T, excl, tok, u, slack):
    """Is u within `slack` of the interval that id `tok` owns in the oracle's CDF (id `excl` removed)?"""
    p = oracle.target_probs(logits_row, T).clone()
    if excl is not None:
        p[excl] = 0.0
    c = torch.cumsum(p, 0) / p.sum()
    lo = float(c[tok - 1]) if tok > 0 else 0.0
    return lo - slack <= u <= float(c[tok]) + slack


def _temperature_for(logits, draft, target=0.5):
    """The largest temperature of a halving ladder at which the drafts' mean accept probability reaches `target`
    (a random-init model is nearly uniform at T = 1; the test wants both acceptances and rejections)."""
    T = 1.0
    while T > 1e-3:
        if not draft or np.mean([float(oracle.target_probs(logits[j], T)[x]) for j, x in enumerate(draft)]) >= target:
            return T
        T /= 2
    return T


@pytest.mark.parametrize("name,ctx,k", [("tiny", 40, 6), ("8b-2l", 300, 9), ("1b-2l", 131, 16), ("8b-2l", 64, 1)])
def test_sampled_acceptance_matches_the_oracle(name, ctx, k):
    shape = synth.SHAPES[name]
    om, gm = make_pair(shape, k_max=max(k, 8), max_ctx=ctx + 64, path=1)
    cache, s, pending = synthetic_context(shape, om, gm, ctx)
    # drafts along the oracle's greedy continuation, so that accept probabilities are sizeable at this temperature
    c, p, draft = cache.clone(), pending, []
    for _ in range(k - 1):
        p = om.greedy_next(p, c)
        draft.append(p)
    logits = om.forward_chunk([pending] + draft, cache.clone())
    T = _temperature_for(logits, draft)
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x5A3B00 + k]))
    slack = 4.0 * LOGIT_MAX_ABS / T / 10      # relative probability error allowed by the logit tolerance
    lens, exact = [], 0
    for trial in range(40):
        u = [float(x) for x in g.random(k).astype(np.float32)]
        u = [min(x, 0.99999994) for x in u]
        l_ref, em_ref = oracle.accept_sampled(logits, draft, T, u)
        res = ts.ts_verify_sampled(gm, [s], [draft], T, u)[0]
        l, em = res.accept_len, list(res.emitted[:res.n_emitted])
        assert res.n_emitted == l + 1 and em[:l] == draft[:l]
        if (l, em) == (l_ref, em_ref):
            exact += 1
        else:
            j = min(l, l_ref)
            if l != l_ref:       # an accept test went the other way: its margin must be small
                pj = float(oracle.target_probs(logits[j], T)[draft[j]])
                assert abs(u[j] - pj) <= slack * pj + 1e-6, f"trial {trial}: accept test {j}: u={u[j]} p={pj}"
            else:                # same length, other sample: the uniform lies next to the id's interval
                excl = draft[l] if l < k - 1 else None
                assert _near_boundary(logits[l], T, excl, em[l], u[k - 1], slack), f"trial {trial}: sample {em[l]}"
        lens.append(l_ref)
    assert exact >= 36                                 # disagreements are the rare case
    if k > 2:
        assert 0 < sum(lens) < 40 * (k - 1)            # both acceptances and rejections occurred
    # commit the last step and check a following greedy step on the resulting cache
    res = ts.ts_verify_sampled(gm, [s], [draft], T, u)[0]
    ts.ts_commit(s, res)
    cache2 = cache.clone()
    om.forward_chunk([pending] + draft[:res.accept_len], cache2)
    nxt = res.emitted[res.accept_len]
    ref2 = om.verify(nxt, [], cache2, want_logits=True)
    res2 = ts.ts_verify(gm, [s], [[]])[0]
    err = np.abs(gm.read_logits(0, 1).astype(np.float64) - ref2["logits"].numpy())
    assert err.max() <= LOGIT_MAX_ABS
    gm.close()


def test_sampled_batch_and_errors():
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, max_batch=2, k_max=8, max_rows=16, max_ctx=256, path=1)
    c0, s0, p0 = synthetic_context(shape, om, gm, 50, stream=0)
    c1, s1, p1 = synthetic_context(shape, om, gm, 17, stream=1)
    d0 = [om.greedy_next(p0, c0.clone()), 100, 101]
    d1 = [om.greedy_next(p1, c1.clone())]
    l0 = om.forward_chunk([p0] + d0, c0.clone())
    l1 = om.forward_chunk([p1] + d1, c1.clone())
    T = _temperature_for(l0, d0[:1])
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x5A3BFF]))
    agree = 0
    for _ in range(20):
        u = [min(float(x), 0.99999994) for x in g.random(6).astype(np.float32)]
        r = ts.ts_verify_sampled(gm, [s0, s1], [d0, d1], T, u)
        want0 = oracle.accept_sampled(l0, d0, T, u[:4])
        want1 = oracle.accept_sampled(l1, d1, T, u[4:])
        agree += (r[0].accept_len, list(r[0].emitted[:r[0].n_emitted])) == want0
        agree += (r[1].accept_len, list(r[1].emitted[:r[1].n_emitted])) == want1
    assert agree >= 36
    with pytest.raises(ts.TsError):
        ts.ts_verify_sampled(gm, [s0], [d0], 0.0, [0.5] * 4)             # temperature must be positive
    with pytest.raises(ts.TsError):
        ts.ts_verify_sampled(gm, [s0], [d0], 1.0, [0.5, 1.0, 0.1, 0.2])  # a uniform outside [0, 1)
    with pytest.raises(ts.TsError) as e:                                   # two children of the root with one token:
        ts.ts_verify_tree_sampled(gm, [s0], [[100, 101, 100]], [[0, 1, 0]], 1.0, [0.5] * 4)   # its weight would be removed twice
    assert e.value.code == -1 and "same token" in str(e.value)
    ts.ts_verify_tree(gm, [s0], [[100, 101, 100]], [[0, 1, 0]])           # (greedy acceptance takes the first of them)
    gm.close()


@pytest.mark.parametrize("name,ctx,n_nodes", [("tiny", 40, 12), ("8b-2l", 300, 24)])
def test_sampled_acceptance_over_a_tree(name, ctx, n_nodes):
    """ts_verify_tree_sampled against the oracle's walk with the same uniforms: path and emitted ids agree in at
    least 90% of the trials (a floating-point decision next to its threshold may fall the other way); every result
    is a root path of the tree followed by one more id; the cache after compaction matches the oracle's rows."""
    shape = synth.SHAPES[name]
    om, gm = make_pair(shape, k_max=max(n_nodes, 8), max_ctx=ctx + 64, path=1)
    cache, s, pending = synthetic_context(shape, om, gm, ctx)
    c, p, truth = cache.clone(), pending, []
    for _ in range(4):
        p = om.greedy_next(p, c)
        truth.append(p)
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x5A3C00 + n_nodes]))
    lg0 = om.forward_chunk([pending], cache.clone())[0]
    second = [int(i) for i in torch.topk(lg0, 3).indices.tolist() if int(i) != truth[0]][:2]   # likely siblings of the truth
    junk = lambda n: [int(t) for t in g.integers(64, shape.vocab, size=n)]
    cands = [[second[0]] + junk(2), truth + junk(2), [second[1]] + junk(1), truth[:2] + junk(3), junk(3)]
    toks, par = oracle.pack_candidates(cands, n_nodes)
    z = [pending] + toks
    logits, k_new, v_new = oracle.forward_tree(om, z, par, cache)
    T = 1.0
    while T > 1e-3 and float(oracle.target_probs(logits[0], T)[truth[0]]) < 0.4:
        T /= 2
    exact, lens = 0, []
    for trial in range(40):
        u = [min(float(x), 0.99999994) for x in g.random(len(z)).astype(np.float32)]
        want_path, want_em = oracle.accept_sampled_tree(logits, z, par, T, u)
        res, paths = ts.ts_verify_tree_sampled(gm, [s], [toks], [par[1:]], T, u)
        r, path = res[0], paths[0]
        em = list(r.emitted[:r.n_emitted])
        assert path[0] == 0 and all(par[path[j]] == path[j - 1] for j in range(1, len(path)))
        assert em[:-1] == [z[c] for c in path[1:]] and r.accept_len == len(path) - 1
        exact += (path, em) == (want_path, want_em)
        lens.append(len(want_path) - 1)
    assert exact >= 36
    assert 0 < sum(lens) and min(lens) < max(lens)              # walks of different lengths occurred
    # commit the last trial if it agreed, and compare the compacted cache with the oracle's rows of that path
    if (path, em) == (want_path, want_em):
        ts.ts_commit(s, r)
        n_new = ctx + len(path)
        for l in range(shape.n_layers):
            k, v = s.export_kv(l, n_new)
            for got, want in ((k, k_new[l]), (v, v_new[l])):
                ref = want[torch.tensor(path)]
                d = (got[ctx:].double() - ref).abs()
                assert bool((d <= 1e-2 + 1e-2 * ref.abs()).all())
    gm.close()
