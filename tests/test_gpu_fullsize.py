"""Full-size parity: every benchmark configuration at its stated size against the float64 oracle, on every logit.

The 8B-shaped decoder at full depth (36 layers, 151 936 ids), all in ONE pass over the layers:

  * C3: batch 1, 8192-token context, k = 32 -- the workload and the launch configuration the benchmark times --
    once per step implementation (one kernel per stage, persistent kernel);
  * a ragged batch of three sessions (8192 / 2500 / 5000 cached tokens, k = 32 / 17 / 64);
  * C5: batch 4, 8192-token contexts, k = 64 (256 rows: two 128-row chunks per weight tile, two row tiles per
    sequence in attention);
  * C4: the benchmark's own 16 ragged sessions (contexts log-uniform over 2k..16k, k uniform in 4..32; about 110k
    cached tokens and 286 rows).

The model is too large to hold twice on the host, so all sides are fed layer by layer from the same seeded
generators: a layer's weights (norm gains 1 + 0.3 N(0,1), so that a gain vector taken from the wrong layer or norm
cannot pass) and the sessions' synthetic context K/V are generated once, loaded into the GPU models, pushed through
the oracle's own layer routine (all sequences of all cases as one batch of independent sequences), and dropped.  The
oracle then applies its head to the final residual rows; each GPU model runs one ordinary `ts_verify`.  Nothing the
oracle consumes comes from the GPU.

The 1B-shaped decoder (C2: 16 layers, 128 256 ids, head_dim 64, 4096-token context, k = 4 / 8 / 16) fits on the host
and goes through the ordinary harness, on both step implementations.
"""
import os
import sys
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from paper_2604_13519_b200 import binding as B
from gpu_util import check_step, make_pair, synthetic_context

pytestmark = pytest.mark.gpu

LAYER_KINDS = dict(wq=B.TS_W_Q, wk=B.TS_W_K, wv=B.TS_W_V, wo=B.TS_W_O, wg=B.TS_W_GATE, wu=B.TS_W_UP,
                   wd=B.TS_W_DOWN, g1=B.TS_W_GAIN1, g2=B.TS_W_GAIN2)
GAIN_SEED = 7


def _c4_sessions():
    """The benchmark's config-4 workload (its generator is the single statement of it)."""
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    _shape, lens, ks = bench.c4_workload()
    return list(zip(lens, ks))


def _model(shape, seqs, path):
    """The benchmark's model configuration for these sequences."""
    lens, ks = [n for n, _ in seqs], [k for _, k in seqs]
    k_max = max(max(ks), 8)
    pages = sum((n + 2 * k_max + 15) // 16 for n in lens) + 8
    return ts.Model(shape, max_pages=pages, max_batch=len(seqs), k_max=k_max, max_rows=max(sum(ks), k_max),
                    max_ctx=max(lens) + 2 * k_max, act_split=True, path=path)


def _extras_at_full_vocabulary(gm, sess, draft, logits):
    """The per-position Top-K and the sampling acceptance on the full 151 936-id vocabulary (37 whole 4096-id slices
    and a ragged one), against the oracle's logits of the same chunk."""
    k = len(draft) + 1
    ts.ts_verify(gm, [sess], [draft], flags=ts.TS_FLAG_WANT_TOPK)
    exact = 0
    for j in range(k):
        ids, vals = ts.ts_last_topk(gm, j)
        want = oracle.topk_lowest(logits[j], ts.TS_TOPK)
        assert len(set(ids)) == ts.TS_TOPK
        for r, i in enumerate(ids):
            assert float(logits[j][i]) >= float(logits[j][want[r]]) - 0.05, f"row {j} rank {r}"
        exact += ids == want
    assert exact >= k // 2        # with 151 936 ids the 8 best lie close together: swaps inside the margin are common
    # sampling acceptance: at a temperature where the greedy token is a coin flip, same uniforms on both sides
    T = 1.0
    while T > 1e-3 and float(oracle.target_probs(logits[0], T).max()) < 0.5:
        T /= 2
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x8B37]))
    agree = 0
    for _ in range(12):
        u = [min(float(x), 0.99999994) for x in g.random(k).astype(np.float32)]
        want = oracle.accept_sampled(logits, draft, T, u)
        r = ts.ts_verify_sampled(gm, [sess], [draft], T, u)[0]
        agree += (r.accept_len, list(r.emitted[:r.n_emitted])) == want
    assert agree >= 10


def test_8b_full_depth_all_configurations():
    shape = synth.SHAPES["8b"]
    assert shape.n_layers == 36
    # the oracle's sequences: (cached tokens, chunk rows); the K/V stream of a sequence is its index here
    seqs = [(8192, 32), (2500, 17), (5000, 64)] + [(8192, 64)] * 4 + _c4_sessions()
    c5, c4 = list(range(3, 7)), list(range(7, len(seqs)))
    # (name, step implementation, sequences): the first two are the benchmark's default workload
    plan = [("c3 batch 1, separate kernels", 1, [0]), ("c3 batch 1, persistent kernel", 2, [0]),
            ("ragged batch of three", 0, [0, 1, 2]), ("c5 batch 4 x k 64", 0, c5), ("c4 sixteen ragged sessions", 0, c4)]
    models = [_model(shape, [seqs[i] for i in idx], path) for _, path, idx in plan]
    sessions = [[ts.Session(gm, None, None) for _ in idx] for gm, (_, _, idx) in zip(models, plan)]

    glob = synth.make_weights(shape, layers=[], gain_seed=GAIN_SEED)              # embedding, LM head, final gain
    for gm in models:
        gm.load_tensor(B.TS_W_EMBED, 0, glob["embed"])
        gm.load_tensor(B.TS_W_LM_HEAD, 0, glob["lm_head"])
        gm.load_tensor(B.TS_W_FINAL_GAIN, 0, glob["gf"].float())

    pending = synth.Vocab(shape.vocab).tool_call
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x8B36]))
    drafts = [[int(t) for t in g.integers(64, shape.vocab, size=k - 1)] for _, k in seqs]
    x = [glob["embed"][torch.tensor([pending] + d)].to(torch.float64) for d in drafts]
    poss = [torch.arange(k) + n for n, k in seqs]
    pos_prev = [torch.arange(n) for n, _ in seqs]

    pool = ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4))
    for l in range(shape.n_layers):
        kv_jobs = [pool.submit(synth.make_synthetic_kv, shape, n, stream=i, layers=[l]) for i, (n, _) in enumerate(seqs)]
        wl = synth.make_weights(shape, layers=[l], with_globals=False, gain_seed=GAIN_SEED)
        for gm in models:
            for n, kind in LAYER_KINDS.items():
                t = wl[f"l{l}.{n}"]
                gm.load_tensor(kind, l, t.float() if n[0] == "g" else t)
        kv = [j.result() for j in kv_jobs]
        for (_, _, idx), ss in zip(plan, sessions):
            for s, i in zip(ss, idx):
                s.import_kv(l, kv[i][0][0], kv[i][1][0])
        om = oracle.OracleModel(shape, wl)
        x, _, _ = om._layer_multi(l, x, poss, [K[0].to(torch.float64) for K, _ in kv], [V[0].to(torch.float64) for _, V in kv],
                                  pos_prev)
        del wl, om, kv, kv_jobs
    pool.shutdown()

    head = oracle.OracleModel(shape, glob)
    refs = []
    for i, d in enumerate(drafts):
        logits = head._head(x[i])
        t = oracle.argmax_lowest(logits)
        n_acc = 0
        while n_acc < len(d) and t[n_acc] == d[n_acc]:
            n_acc += 1
        refs.append(dict(logits=logits, argmax=t, accept_len=n_acc, emitted=d[:n_acc] + [t[n_acc]]))

    failures = []
    for (name, path, idx), gm, ss in zip(plan, models, sessions):
        for s, i in zip(ss, idx):
            s.set_cache(seqs[i][0], pending)
        res = ts.ts_verify(gm, ss, [drafts[i] for i in idx])
        row0, worst_max, worst_mean = 0, 0.0, 0.0
        for r, i in zip(res, idx):
            k = seqs[i][1]
            got = gm.read_logits(row0, k)
            where = f"8b x 36 layers, {name}, sequence {i} (ctx {seqs[i][0]}, k {k})"
            try:
                assert np.isfinite(got).all(), where
                mx, mean = check_step(r, got, refs[i], where=where)
                worst_max, worst_mean = max(worst_max, mx), max(worst_mean, mean)
            except AssertionError as e:
                failures.append(str(e))
            row0 += k
        print(f"8b x 36 layers, {name}: worst sequence logits max-abs {worst_max:.3e}, mean-abs {worst_mean:.3e}")
        if path == 1 and not failures:
            _extras_at_full_vocabulary(gm, ss[0], drafts[idx[0]], refs[idx[0]]["logits"])
        gm.close()
    assert not failures, "\n".join(failures)


@pytest.mark.parametrize("path", [pytest.param(1, id="separate"), pytest.param(2, id="fused")])
def test_1b_full_depth(path):
    """C2 at its stated size: 16 layers, width 2048, heads of 64, 128 256 ids, 4096 cached tokens, k = 4, 8, 16 on the
    same context (the steps are not committed, so each sees the imported cache)."""
    shape = synth.SHAPES["1b"]
    assert (shape.n_layers, shape.vocab) == (16, 128256)
    w = synth.make_weights(shape, gain_seed=GAIN_SEED)
    om, gm = make_pair(shape, k_max=16, max_ctx=4096 + 64, weights=w, path=path)
    cache, s, pending = synthetic_context(shape, om, gm, 4096)
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x1B16]))
    draft = [int(t) for t in g.integers(64, shape.vocab, size=15)]
    for k in (4, 8, 16):
        ref = om.verify(pending, draft[:k - 1], cache.clone(), want_logits=True)
        res = ts.ts_verify(gm, [s], [draft[:k - 1]])[0]
        mx, mean = check_step(res, gm.read_logits(0, k), ref, f"1b x 16 layers, path {path}, ctx 4096, k {k}")
        print(f"1b x 16 layers, path {path}, k {k}: logits max-abs {mx:.3e}, mean-abs {mean:.3e}")
    gm.close()
