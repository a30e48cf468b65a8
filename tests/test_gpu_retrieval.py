"""ts_topk_cosine against the oracle's Top-K (Eq. 3), and the hidden state it takes as the query against the
oracle's final-norm hidden state of the same row."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from gpu_util import make_pair, synthetic_context

pytestmark = pytest.mark.gpu


def _hidden_store(n, d, seed, q=None):
    """Seeded N(0,1) hidden states rounded to bf16; a few entries planted near the query."""
    g = np.random.Generator(np.random.Philox(key=[260413519, 0xC05 + seed]))
    H = torch.from_numpy(g.standard_normal((n, d), dtype=np.float32))
    if q is not None:
        for rank, j in enumerate((n // 3, 7, n - 1, n // 2)):
            H[j] = q * (1.5 + rank) + torch.from_numpy(g.standard_normal(d, dtype=np.float32)) * (0.2 + 0.3 * rank) * float(q.std())
    return H.to(torch.bfloat16)


@pytest.mark.parametrize("n,d,K", [(1000, 256, 10), (20011, 4096, 10), (37, 2048, 37), (5000, 4096, 64)])
def test_topk_matches_oracle(n, d, K):
    shape = synth.SHAPES[{256: "tiny", 2048: "1b-2l", 4096: "8b-2l"}[d]]
    g = np.random.Generator(np.random.Philox(key=[260413519, 0xC0500 + n]))
    q = torch.from_numpy(g.standard_normal(d, dtype=np.float32))
    H = _hidden_store(n, d, n, q)
    H[min(n - 1, 11)] = 0                                               # a zero vector must rank last
    H[min(n - 1, 12)] = H[min(n - 1, 5)]                                # an exact tie
    gm = ts.Model(shape, max_pages=8, max_batch=1, k_max=8, max_rows=8, max_ctx=64, act_split=True, path=1)
    idx, sc = ts.ts_topk_cosine(gm, H.cuda(), K, query=q.cuda())
    ref_idx, ref_sc = oracle.topk_cosine(H, q, K)
    assert np.allclose(sc, ref_sc, rtol=0, atol=2e-5)
    s_all = oracle.cosine_scores(H, q)
    for j in range(K):
        if idx[j] != ref_idx[j]:     # only where two oracle scores are closer than the fp32 arithmetic resolves
            assert abs(float(s_all[idx[j]]) - ref_sc[j]) < 2e-5, (j, idx[j], ref_idx[j])
    assert len(set(idx)) == K
    if K == n:
        assert idx[-1] == 11 and sc[-1] == -2.0
    assert idx[:4] == ref_idx[:4] == [n // 3, 7, n - 1, n // 2] or K < 4 or n < 40
    gm.close()


def test_query_from_the_last_step_is_the_final_hidden_state():
    shape = synth.SHAPES["8b-2l"]
    om, gm = make_pair(shape, k_max=8, max_ctx=256, path=1)
    cache, s, pending = synthetic_context(shape, om, gm, 100)
    draft = [200, 300, 400]
    probe = {}
    om.forward_chunk([pending] + draft, cache.clone(), probe=probe)
    hx = oracle.rmsnorm(probe["x_final"], om.w["gf"], shape.rms_eps)          # the LM head's input, [4, d]
    ts.ts_verify(gm, [s], [draft])
    for row in (0, 3):
        got = ts.ts_last_hidden(gm, row)
        assert np.abs(got.astype(np.float64) - hx[row].numpy()).max() <= 2e-2 * float(hx[row].abs().max())
    # the library's own query (row 0) ranks a store like the oracle's hidden state does
    H = _hidden_store(3000, shape.d_model, 1, hx[0].float())
    idx, sc = ts.ts_topk_cosine(gm, H.cuda(), 10, query=None, row=0)
    ref_idx, ref_sc = oracle.topk_cosine(H, hx[0], 10)
    assert idx[:4] == ref_idx[:4]
    assert np.allclose(sc[:4], ref_sc[:4], rtol=0, atol=5e-3)
    with pytest.raises(ts.TsError):
        ts.ts_topk_cosine(gm, H.cuda(), 0)
    gm.close()


def test_algorithm_1_retrieval_end_to_end():
    """Algorithm 1 driven from the library's own datastore H = {(h_j, y_j)}: N historical invocations inserted with the
    hidden state of their question's last token (device-to-device, into a matrix the test owns); then, per query,
    h_x -> Top-10 -> I_k installed on the session -> drafts (the schema draft's tool guess and the suffix match, both
    restricted to I_k) equal to the oracle's, which ranks its own float64 hidden states rounded to bf16."""
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=16, max_ctx=256, path=1)
    schema = synth.make_schema(shape.vocab, 8)
    inv = synth.make_datastore(schema, 40)
    sc = ts.Schema(schema.vocab, schema.tools)
    questions = [synth.make_context(shape.vocab, 20 + i % 7, stream=100 + i) for i in range(len(inv))]
    H = torch.zeros(len(inv) + 2, shape.d_model, dtype=torch.bfloat16, device="cuda")
    st_c, st_o, hs_o = ts.Datastore(len(schema.tools)), oracle.Datastore(len(schema.tools)), oracle.HiddenStore()
    with pytest.raises(ts.TsError) as e:
        st_c.add_hidden(gm, 0, inv[0][1], inv[0][0])           # nothing attached yet
    assert e.value.code == -2
    st_c.attach_hidden(H)

    def final_hidden(prompt):
        cache, pending = oracle.prefill(om, prompt)
        probe = {}
        om.forward_chunk([pending], cache, probe=probe)
        return oracle.rmsnorm(probe["x_final"], om.w["gf"], shape.rms_eps)[0]

    for (tid, toks), q in zip(inv, questions):
        s = ts.Session(gm, None, None)
        ts.ts_prefill(gm, s, q)
        ts.ts_verify(gm, [s], [[]])                             # row 0 = the question's last token
        st_c.add_hidden(gm, 0, toks, tid)
        s.close()
        st_o.add(toks, tid)
        hs_o.add(final_hidden(q))
    with pytest.raises(ts.TsError) as e:
        st_c.add(inv[0][1], inv[0][0])                          # an entry without its hidden state
    assert e.value.code == -2
    torch.cuda.synchronize()
    want_rows = torch.stack(hs_o.rows).float()
    got_rows = H[:len(inv)].float().cpu()
    assert (got_rows - want_rows).abs().max() <= 2e-2 * want_rows.abs().max()
    assert float(H[len(inv):].abs().max()) == 0.0              # rows of entries that do not exist were not written

    exact = 0
    for trial, j_star in enumerate((5, 17, 33, 0)):
        q = list(questions[j_star])
        q[2 + trial] = (q[2 + trial] + 1) % shape.vocab         # the stored question, one token changed
        s = ts.Session(gm, sc, st_c)
        ts.ts_prefill(gm, s, q)
        ts.ts_verify(gm, [s], [[]])
        idx, score = ts.ts_session_retrieve(gm, s, 10)
        h_x = final_hidden(q)
        ref_idx, ref_score = hs_o.retrieve(h_x, 10)
        assert idx[0] == ref_idx[0] == j_star
        assert np.allclose(score, ref_score, rtol=0, atol=1e-2)
        s_all = oracle.cosine_scores(torch.stack(hs_o.rows), h_x)
        for r in range(10):       # a rank may differ only between entries whose oracle scores nearly tie
            assert idx[r] == ref_idx[r] or abs(float(s_all[idx[r]]) - ref_score[r]) < 1e-2, (r, idx, ref_idx)
        exact += idx == ref_idx
        s.set_ranks(ref_idx)                                    # (same candidate order on both sides from here on)
        d = oracle.Drafter(schema, st_o, ranks=ref_idx)
        d.feed_prompt(q)
        # the schema draft: the tool is guessed from the best-ranked candidate
        assert ts.ts_draft(s, 15) == d.draft(15)
        # the suffix match, restricted to I_k: continue with the opening of the third-ranked invocation
        toks = st_o.entries[ref_idx[2]]
        ts.ts_verify(gm, [s], [toks[:7]])
        ts.ts_commit_forced(s, toks[:8])
        d.commit(toks[:8], schema.vocab.eos, 10 ** 6)
        got, want = ts.ts_draft(s, 15), d.draft(15)
        assert got == want and want[1] == 2 and len(want[0]) > 0
        # an invocation outside I_k is never matched, although the whole store would match it
        outside = next(c for c in range(len(inv)) if c not in ref_idx and len(st_o.entries[c]) > 9)
        s2 = ts.Session(gm, sc, st_c)
        ts.ts_prefill(gm, s2, q)
        ts.ts_verify(gm, [s2], [st_o.entries[outside][:7]])
        s2.set_ranks(ref_idx)
        ts.ts_commit_forced(s2, st_o.entries[outside][:8])
        d2 = oracle.Drafter(schema, st_o, ranks=ref_idx)
        d2.feed_prompt(q)
        d2.commit(st_o.entries[outside][:8], schema.vocab.eos, 10 ** 6)
        assert ts.ts_draft(s2, 15) == d2.draft(15)
        s.close(); s2.close()
    assert exact >= 3
    gm.close()
