"""General speculative drafting for the open-ended states: the per-position Top-K of the verify logits
(TS_FLAG_WANT_TOPK) against the oracle's, the successor lists the library builds from it, and the draft ->
verify -> commit loop with context matches and recycled-successor trees following the oracle's trajectory."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from gpu_util import make_pair, synthetic_context, LOGIT_MAX_ABS, GAP

pytestmark = pytest.mark.gpu


def _check_topk(ids, vals, logits_row, where):
    """ids are distinct, and the j-th pick is worth the oracle's j-th value up to the near-tie margin."""
    want = oracle.topk_lowest(logits_row, ts.TS_TOPK)
    assert len(set(ids)) == ts.TS_TOPK, where
    for j, (i, v) in enumerate(zip(ids, vals)):
        assert abs(v - float(logits_row[i])) <= LOGIT_MAX_ABS, where
        assert float(logits_row[i]) >= float(logits_row[want[j]]) - GAP, f"{where}: rank {j}"
    return ids == want


@pytest.mark.parametrize("name,ctx,k", [("tiny", 40, 8), ("8b-2l", 300, 32), ("1b-2l", 131, 5)])
def test_per_position_topk(name, ctx, k):
    shape = synth.SHAPES[name]
    om, gm = make_pair(shape, k_max=max(k, 8), max_ctx=ctx + 64, path=1)
    cache, s, pending = synthetic_context(shape, om, gm, ctx)
    s.enable_general_sd()
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x70B00 + k]))
    draft = [int(t) for t in g.integers(64, shape.vocab, size=k - 1)]
    logits = om.forward_chunk([pending] + draft, cache.clone())
    res = ts.ts_verify(gm, [s], [draft], flags=ts.TS_FLAG_WANT_TOPK)[0]
    exact = 0
    for j in range(k):
        ids, vals = ts.ts_last_topk(gm, j)
        exact += _check_topk(ids, vals, logits[j], f"{name} row {j}")
        assert ids[0] == res.argmax[j]
        assert s.successors(([pending] + draft)[j]) is not None
    assert exact >= k - 2                                   # near-ties inside the top 8 are the rare case
    # the lists the session now holds are those rows' Top-K (the last row that fed a token wins)
    chunk = [pending] + draft
    for t in set(chunk):
        j = max(i for i, z in enumerate(chunk) if z == t)
        assert s.successors(t) == ts.ts_last_topk(gm, j)[0]
    # without the flag nothing is refreshed, and asking for the Top-K is an error
    ts.ts_verify(gm, [s], [draft])
    with pytest.raises(ts.TsError):
        ts.ts_last_topk(gm, 0)
    gm.close()


def test_general_sd_loop_follows_the_oracle():
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=20, max_ctx=512, path=1)
    schema = synth.make_schema(shape.vocab, 8)
    v = schema.vocab
    prompt = synth.make_context(shape.vocab, 120)[:-1] + [77]          # no tool call: q_o throughout
    sc = ts.Schema(schema.vocab, schema.tools)
    d = oracle.Drafter(schema, oracle.Datastore(len(schema.tools)), general_sd=True)
    d.feed_prompt(prompt)
    cache, pending = oracle.prefill(om, prompt)
    s = ts.Session(gm, sc, None, max_new_tokens=48)
    s.enable_general_sd()
    ts.ts_prefill(gm, s, prompt)
    y_ref = oracle.vanilla_greedy(om, schema, prompt, v.eos, 48)
    sources, accepted = [], []
    for step in range(48):
        wt, wp, wsrc = d.draft_tree(20)
        gt, gp, gsrc = ts.ts_draft_tree(s, 20)
        assert (gt, gp, gsrc) == (wt, wp[1:], wsrc), f"step {step}"
        sources.append(wsrc)
        n0 = cache.length
        ref = oracle.verify_tree(om, pending, wt, wp, cache, want_logits=True)
        res, paths = ts.ts_verify_tree(gm, [s], [gt], [gp], flags=ts.TS_FLAG_WANT_TOPK)
        chunk = [pending] + wt
        rows = [oracle.topk_lowest(ref["logits"][j], oracle.TOPK) for j in range(len(chunk))]
        for j in range(len(chunk)):
            ids, vals = ts.ts_last_topk(gm, j)
            _check_topk(ids, vals, ref["logits"][j], f"step {step} row {j}")
        d.update_successors(chunk, rows)
        for t in set(chunk):                                # keep both sides on the oracle's lists
            s.set_successors(t, d.successors[t])
        if paths[0] != ref["path"] or list(res[0].emitted[:res[0].n_emitted]) != ref["emitted"]:
            j = ref["path"][min(len(paths[0]), len(ref["path"])) - 1]
            assert oracle.top2_gap(ref["logits"][j]) < GAP
            break
        used, fin = d.commit(ref["emitted"], v.eos, 48)
        cache.truncate(n0 + used)
        ts.ts_commit(s, res[0])
        pending = ref["emitted"][used - 1]
        assert (s.state().cache_len, s.state().pending) == (cache.length, pending)
        accepted.append(ref["accept_len"])
        if fin:
            assert s.output() == d.y == y_ref[:len(d.y)]
            break
    assert 4 in sources and sources[0] == 0
    gm.close()
