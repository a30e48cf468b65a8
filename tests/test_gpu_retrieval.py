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
