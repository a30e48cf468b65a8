"""Helpers for the GPU parity tests: build both sides from the same seeded inputs and compare."""
import numpy as np
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts

LOGIT_MAX_ABS = 3e-2     # tolerance on logits against the float64 oracle
LOGIT_MEAN_ABS = 3e-3
GAP = 0.05               # integer results may differ only where the oracle's top-2 gap is below this


GAIN_SEED = 7            # norm gains 1 + 0.3 N(0,1): a gain vector taken from the wrong layer or norm cannot pass


def make_pair(shape, max_batch=1, k_max=8, max_rows=None, max_ctx=1024, max_pages=None, act_split=True,
              weights=None, path=0):
    w = weights if weights is not None else synth.make_weights(shape, gain_seed=GAIN_SEED)
    om = oracle.OracleModel(shape, w)
    max_rows = max_rows or max_batch * k_max
    max_pages = max_pages or max_batch * ((max_ctx + 15) // 16)
    gm = ts.Model(shape, max_pages=max_pages, max_batch=max_batch, k_max=k_max, max_rows=max_rows,
                  max_ctx=max_ctx, act_split=act_split, path=path)
    gm.load_weights(w)
    return om, gm


def synthetic_context(shape, om, gm, length, stream=0, schema=None, store=None, n_cap=32, pending=None):
    """A sequence whose cache holds `length` tokens of seeded synthetic K/V on both sides."""
    K, V = synth.make_synthetic_kv(shape, length, stream=stream)
    cache = om.new_cache()
    cache.import_kv(K, V)
    s = ts.Session(gm, schema, store, n_cap=n_cap)
    for l in range(shape.n_layers):
        s.import_kv(l, K[l], V[l])
    if pending is None:
        pending = synth.Vocab(shape.vocab).tool_call
    s.set_cache(length, pending)
    return cache, s, pending


def check_step(res, logits_gpu, ref, where=""):
    """res: ts_verify_result; logits_gpu: [k, V] float32; ref: oracle verify dict with logits."""
    lo = ref["logits"].numpy()
    err = np.abs(logits_gpu.astype(np.float64) - lo)
    assert err.max() <= LOGIT_MAX_ABS, f"{where}: logits max-abs {err.max():.3e}"
    assert err.mean() <= LOGIT_MEAN_ABS, f"{where}: logits mean-abs {err.mean():.3e}"
    k = lo.shape[0]
    gaps = [oracle.top2_gap(ref["logits"][j]) for j in range(k)]
    for j in range(k):
        if gaps[j] >= GAP:
            assert res.argmax[j] == ref["argmax"][j], f"{where}: argmax row {j}"
        else:   # near-tie: the GPU's choice must still be one of the oracle's top two
            top2 = torch.topk(ref["logits"][j], 2).indices.tolist()
            assert res.argmax[j] in top2, f"{where}: argmax row {j} outside the oracle's top two"
    # accepted length and emitted ids: exact unless a row up to the first difference is a near-tie
    l_ref = ref["accept_len"]
    first_diff = next((j for j in range(k) if res.argmax[j] != ref["argmax"][j]), None)
    if first_diff is None or first_diff > l_ref:
        assert res.accept_len == l_ref, f"{where}: accept_len {res.accept_len} vs {l_ref}"
        assert list(res.emitted[:res.n_emitted]) == ref["emitted"], f"{where}: emitted ids"
    else:
        assert gaps[first_diff] < GAP
    assert res.n_emitted == res.accept_len + 1
    return float(err.max()), float(err.mean())
