"""ts_verify_tree against the oracle's tree verification (Appendix A.1; Algorithm 1: PackDraftsAsTree,
Verification, SelectLongestAcceptedPrefix): logits of every node, the accepted path, the emitted ids,
the cache after compaction, and a following ordinary step on the compacted cache."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from gpu_util import make_pair, synthetic_context, LOGIT_MAX_ABS, LOGIT_MEAN_ABS, GAP

pytestmark = pytest.mark.gpu


def _greedy(om, cache, pending, n):
    """The oracle's next n greedy tokens (on a copy of the cache)."""
    c, p, out = cache.clone(), pending, []
    for _ in range(n):
        p = om.greedy_next(p, c)
        out.append(p)
    return out


def _candidates(g, vocab, truth, n_nodes):
    """Candidate chains that contain the true continuation among wrong branches; packed to n_nodes."""
    def junk(n):
        return [int(t) for t in g.integers(64, vocab, size=n)]
    cands = [truth[:2] + junk(2), truth + junk(4), junk(5), truth[:1] + junk(3), junk(2)]
    while True:
        toks, par = oracle.pack_candidates(cands, n_nodes)
        if len(par) >= n_nodes:
            return toks, par
        cands.append(truth[:int(g.integers(0, len(truth) + 1))] + junk(int(g.integers(1, 9))))


def _check_tree(res, path, logits_gpu, ref, where):
    lo = ref["logits"].numpy()
    err = np.abs(logits_gpu.astype(np.float64) - lo)
    assert err.max() <= LOGIT_MAX_ABS, f"{where}: logits max-abs {err.max():.3e}"
    assert err.mean() <= LOGIT_MEAN_ABS, f"{where}: logits mean-abs {err.mean():.3e}"
    k = lo.shape[0]
    gaps = [oracle.top2_gap(ref["logits"][j]) for j in range(k)]
    for j in range(k):
        if gaps[j] >= GAP:
            assert res.argmax[j] == ref["argmax"][j], f"{where}: argmax node {j}"
        else:
            assert res.argmax[j] in torch.topk(ref["logits"][j], 2).indices.tolist(), f"{where}: node {j}"
    # the walk may differ only from a node on the oracle's path whose top two logits nearly tie
    same = path == ref["path"] and list(res.emitted[:res.n_emitted]) == ref["emitted"]
    if not same:
        common = 0
        while common < min(len(path), len(ref["path"])) and path[common] == ref["path"][common]:
            common += 1
        assert common >= 1 and gaps[ref["path"][common - 1]] < GAP, f"{where}: path {path} vs {ref['path']}"
    assert res.accept_len == len(path) - 1 and res.n_emitted == res.accept_len + 1
    return same


def _check_cache(shape, sess, cache, n_tokens, first, where):
    """Cache rows [first, n_tokens) of every layer against the oracle's (fp16 storage on the GPU)."""
    for l in range(shape.n_layers):
        k, v = sess.export_kv(l, n_tokens)
        for got, want, nm in ((k, cache.k[l], "K"), (v, cache.v[l], "V")):
            d = (got[first:].double() - want[first:n_tokens]).abs()
            tol = 1e-2 + 1e-2 * want[first:n_tokens].abs()
            assert bool((d <= tol).all()), f"{where}: layer {l} {nm} rows differ by {float(d.max()):.3e}"


@pytest.mark.parametrize("name,ctx,n_nodes", [("tiny", 40, 8), ("1b-2l", 131, 16), ("8b-2l", 700, 64),
                                              ("8b-2l", 2048, 33), ("8b-2l", 9, 20)])
def test_tree_single(name, ctx, n_nodes):
    shape = synth.SHAPES[name]
    om, gm = make_pair(shape, k_max=max(n_nodes, 8), max_ctx=ctx + 160, path=1)
    cache, s, pending = synthetic_context(shape, om, gm, ctx)
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x7EE00 + n_nodes]))
    for step in range(2):
        truth = _greedy(om, cache, pending, 4)
        toks, par = _candidates(g, shape.vocab, truth, n_nodes)
        n0 = cache.length
        ref = oracle.verify_tree(om, pending, toks, par, cache, want_logits=True)
        assert ref["accept_len"] >= 4                                  # the true branch is walked
        res, paths = ts.ts_verify_tree(gm, [s], [toks], [par[1:]])
        where = f"{name} ctx={ctx} nodes={n_nodes} step {step}"
        same = _check_tree(res[0], paths[0], gm.read_logits(0, n_nodes), ref, where)
        if not same:
            break                                                      # permitted near-tie: trajectories part
        ts.ts_commit(s, res[0])
        assert s.state().cache_len == cache.length == n0 + ref["accept_len"] + 1
        _check_cache(shape, s, cache, cache.length, n0, where)
        pending = ref["emitted"][-1]
        assert s.state().pending == pending
    else:
        # an ordinary chain step on the compacted cache
        draft = _greedy(om, cache, pending, 3)
        ref2 = om.verify(pending, draft, cache, want_logits=True)
        res2 = ts.ts_verify(gm, [s], [draft])[0]
        err = np.abs(gm.read_logits(0, 4).astype(np.float64) - ref2["logits"].numpy())
        assert err.max() <= LOGIT_MAX_ABS and err.mean() <= LOGIT_MEAN_ABS
        assert res2.accept_len == ref2["accept_len"] == 3 or min(oracle.top2_gap(ref2["logits"][j]) for j in range(4)) < GAP
    gm.close()


def test_tree_batch_of_two_and_chain_equivalence():
    shape = synth.SHAPES["8b-2l"]
    om, gm = make_pair(shape, max_batch=2, k_max=32, max_rows=64, max_ctx=1400, path=1)
    c0, s0, p0 = synthetic_context(shape, om, gm, 1200, stream=0)
    c1, s1, p1 = synthetic_context(shape, om, gm, 333, stream=1)
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x7EE00 + 2]))
    # a chain given as a tree reproduces ts_verify bit for bit (same kernels, same inputs)
    chain = [int(t) for t in g.integers(64, shape.vocab, size=11)]
    ts.ts_verify(gm, [s0], [chain])
    a = gm.read_logits(0, 12).copy()
    ts.ts_verify_tree(gm, [s0], [chain], [list(range(11))])
    assert np.array_equal(a, gm.read_logits(0, 12))
    # two sequences, different trees, one call
    t0, par0 = _candidates(g, shape.vocab, _greedy(om, c0, p0, 4), 32)
    t1, par1 = _candidates(g, shape.vocab, _greedy(om, c1, p1, 4), 19)
    r0 = oracle.verify_tree(om, p0, t0, par0, c0, want_logits=True)
    r1 = oracle.verify_tree(om, p1, t1, par1, c1, want_logits=True)
    res, paths = ts.ts_verify_tree(gm, [s0, s1], [t0, t1], [par0[1:], par1[1:]])
    ok0 = _check_tree(res[0], paths[0], gm.read_logits(0, 32), r0, "batch seq 0")
    ok1 = _check_tree(res[1], paths[1], gm.read_logits(32, 19), r1, "batch seq 1")
    for ok, s, c, r, n0 in ((ok0, s0, c0, res[0], 1200), (ok1, s1, c1, res[1], 333)):
        if ok:
            ts.ts_commit(s, r)
            _check_cache(shape, s, c, c.length, n0, "batch")
    gm.close()


def test_tree_argument_errors():
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=8, max_ctx=128, path=1)
    cache, s, pending = synthetic_context(shape, om, gm, 20)
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify_tree(gm, [s], [[100, 101, 102]], [[0, 2, 1]])       # parent after its child
    assert e.value.code == -1
    with pytest.raises(ts.TsError):
        ts.ts_verify_tree(gm, [s], [[100, 101]], [[0, -1]])               # a second root
    res, paths = ts.ts_verify_tree(gm, [s], [[]], [[]])                   # no drafts: one vanilla step
    assert res[0].accept_len == 0 and paths[0] == [0]
    assert res[0].emitted[0] == om.greedy_next(pending, cache.clone()) or \
        oracle.top2_gap(om.forward_chunk([pending], cache.clone())[0]) < GAP
    gm.close()
    om2, gm2 = make_pair(shape, k_max=8, max_ctx=128, path=2)
    _, s2, _ = synthetic_context(shape, om2, gm2, 20)
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify_tree(gm2, [s2], [[100]], [[0]])
    assert e.value.code == -8
    gm2.close()


def test_tree_decode_loop_follows_the_oracle():
    """Algorithm 1's loop with candidate trees on the tiny decoder: ts_draft_tree -> ts_verify_tree ->
    ts_commit against the oracle's trajectory, real prefill on both sides, self-history in the datastore
    so that retrieved branches are accepted fully and partially."""
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=24, max_ctx=512, path=1)
    schema = synth.make_schema(shape.vocab, 8)
    inv = synth.make_datastore(schema, 64)
    v = schema.vocab
    prompt = synth.make_context(shape.vocab, 200)
    y_ref = oracle.vanilla_greedy(om, schema, prompt, v.eos, 60)
    bad = list(y_ref)
    for p in (9, 17, 22, 40):
        bad[p] = (bad[p] + 1) % shape.vocab
    inv = inv + [(-1, bad), (-1, y_ref), (-1, y_ref[:30] + bad[30:])]
    st_o, st_c = oracle.Datastore(len(schema.tools)), ts.Datastore(len(schema.tools))
    for tid, toks in inv:
        st_o.add(toks, tid)
        st_c.add(toks, tid)
    sc = ts.Schema(schema.vocab, schema.tools)
    d = oracle.Drafter(schema, st_o)
    d.feed_prompt(prompt)
    cache, pending = oracle.prefill(om, prompt)
    s = ts.Session(gm, sc, st_c, max_new_tokens=60)
    ts.ts_prefill(gm, s, prompt)
    accepted, branched = [], 0
    for step in range(30):
        wt, wp, wsrc = d.draft_tree(24)
        gt, gp, gsrc = ts.ts_draft_tree(s, 24)
        assert (gt, gp, gsrc) == (wt, wp[1:], wsrc)
        branched += len(set(wp)) < len(wp)
        n0 = cache.length
        ref = oracle.verify_tree(om, pending, wt, wp, cache, want_logits=True)
        res, paths = ts.ts_verify_tree(gm, [s], [gt], [gp])
        same = _check_tree(res[0], paths[0], gm.read_logits(0, len(wt) + 1), ref, f"loop step {step}")
        if not same:
            break                                          # permitted near-tie: the trajectories part
        used, fin = d.commit(ref["emitted"], v.eos, 60)
        cache.truncate(n0 + used)
        ts.ts_commit(s, res[0])
        pending = ref["emitted"][used - 1]
        info = s.state()
        assert (info.cache_len, info.pending, bool(info.finished)) == (cache.length, pending, fin)
        accepted.append(ref["accept_len"])
        if fin:
            break
    else:
        raise AssertionError("the generation did not finish in 30 steps")
    if same:
        assert s.output() == d.y == y_ref[:len(d.y)]
        assert max(accepted) >= 8 and branched >= 1
    gm.close()
