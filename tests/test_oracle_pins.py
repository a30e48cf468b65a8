"""Pins for the transformer oracle: each test checks it against something other than itself
(library routines it does not call, closed forms, invariants the paper states, brute force)."""
import math

import pytest
import torch
import torch.nn.functional as F

import oracle
import synth
from oracle.transformer import F64


def _small_shape(**kw):
    base = dict(name="pin", n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16,
                d_ffn=128, vocab=512, rope_theta=10000.0, rms_eps=1e-5)
    base.update(kw)
    return synth.ModelShape(**base)


def _rand_weights(shape, seed=0, std=0.08, random_gains=True):
    w = synth.make_weights(shape, seed=seed)
    g = torch.Generator().manual_seed(seed)
    for k in list(w):
        if w[k].dim() == 2:       # larger std so that attention is far from uniform
            w[k] = (w[k].float() * (std / 0.02)).to(torch.bfloat16)
        elif random_gains:
            w[k] = (1.0 + 0.3 * torch.randn(w[k].shape, generator=g)).float()
    return w


# ---- library-routine pins ----------------------------------------------------------------------
def test_rmsnorm_matches_torch():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(5, 96, generator=g, dtype=F64) * 3
    gain = torch.randn(96, generator=g, dtype=F64)
    ref = F.rms_norm(x, (96,), weight=gain, eps=1e-5)
    assert torch.allclose(oracle.rmsnorm(x, gain, 1e-5), ref, rtol=0, atol=1e-12)


def test_swiglu_matches_torch():
    g = torch.Generator().manual_seed(2)
    a, b = torch.randn(7, 33, generator=g, dtype=F64) * 4, torch.randn(7, 33, generator=g, dtype=F64)
    assert torch.allclose(oracle.swiglu(a, b), F.silu(a) * b, rtol=0, atol=1e-12)


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (4, 2), (8, 1)])
def test_attention_matches_sdpa(Hq, Hkv):
    g = torch.Generator().manual_seed(3)
    Tk, Tq, hd = 19, 5, 16
    q = torch.randn(Tq, Hq, hd, generator=g, dtype=F64)
    k = torch.randn(Tk, Hkv, hd, generator=g, dtype=F64)
    v = torch.randn(Tk, Hkv, hd, generator=g, dtype=F64)
    q_pos = torch.arange(Tk - Tq, Tk)
    k_pos = torch.arange(Tk)
    out = oracle.attention(q, k, v, q_pos, k_pos)
    rep = Hq // Hkv
    kk = k.repeat_interleave(rep, dim=1).permute(1, 0, 2)
    vv = v.repeat_interleave(rep, dim=1).permute(1, 0, 2)
    mask = k_pos[None, :] <= q_pos[:, None]
    ref = F.scaled_dot_product_attention(q.permute(1, 0, 2), kk, vv, attn_mask=mask)
    assert torch.allclose(out, ref.permute(1, 0, 2), rtol=0, atol=1e-12)


def test_attention_brute_force_loops():
    g = torch.Generator().manual_seed(4)
    Tk, Tq, Hq, Hkv, hd = 6, 3, 4, 2, 4
    q = torch.randn(Tq, Hq, hd, generator=g, dtype=F64)
    k = torch.randn(Tk, Hkv, hd, generator=g, dtype=F64)
    v = torch.randn(Tk, Hkv, hd, generator=g, dtype=F64)
    q_pos, k_pos = torch.arange(3, 6), torch.arange(6)
    out = oracle.attention(q, k, v, q_pos, k_pos)
    for t in range(Tq):
        for h in range(Hq):
            kh = h // (Hq // Hkv)
            ws = []
            for j in range(Tk):
                if j <= int(q_pos[t]):
                    ws.append(math.exp(sum(float(q[t, h, d]) * float(k[j, kh, d])
                                           for d in range(hd)) / math.sqrt(hd)))
                else:
                    ws.append(0.0)
            z = sum(ws)
            for d in range(hd):
                ref = sum(ws[j] / z * float(v[j, kh, d]) for j in range(Tk))
                assert abs(float(out[t, h, d]) - ref) < 1e-12


def test_whole_forward_matches_hf_llama():
    """The full-recompute driver against Hugging Face's Llama implementation (same recipe:
    pre-norm, RMSNorm, rotate-half RoPE, GQA, SwiGLU, untied head) loaded with the same weights."""
    tr = pytest.importorskip("transformers")
    s = _small_shape()
    w = _rand_weights(s, seed=5)
    cfg = tr.LlamaConfig(hidden_size=s.d_model, num_attention_heads=s.n_q_heads,
                         num_key_value_heads=s.n_kv_heads, head_dim=s.head_dim,
                         intermediate_size=s.d_ffn, vocab_size=s.vocab,
                         num_hidden_layers=s.n_layers, rms_norm_eps=s.rms_eps,
                         rope_theta=s.rope_theta, tie_word_embeddings=False, attention_bias=False,
                         mlp_bias=False, max_position_embeddings=512)
    hf = tr.LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"],
          "model.norm.weight": w["gf"]}
    for l in range(s.n_layers):
        p = f"model.layers.{l}."
        sd[p + "self_attn.q_proj.weight"] = w[f"l{l}.wq"]
        sd[p + "self_attn.k_proj.weight"] = w[f"l{l}.wk"]
        sd[p + "self_attn.v_proj.weight"] = w[f"l{l}.wv"]
        sd[p + "self_attn.o_proj.weight"] = w[f"l{l}.wo"]
        sd[p + "mlp.gate_proj.weight"] = w[f"l{l}.wg"]
        sd[p + "mlp.up_proj.weight"] = w[f"l{l}.wu"]
        sd[p + "mlp.down_proj.weight"] = w[f"l{l}.wd"]
        sd[p + "input_layernorm.weight"] = w[f"l{l}.g1"]
        sd[p + "post_attention_layernorm.weight"] = w[f"l{l}.g2"]
    missing = hf.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [m for m in missing.missing_keys if "rotary" not in m]
    toks = [int(x) for x in torch.randint(0, s.vocab, (23,), generator=torch.Generator().manual_seed(6))]
    with torch.no_grad():
        ref = hf(torch.tensor([toks])).logits[0]
    out = oracle.OracleModel(s, w).forward_full(toks)
    assert float(ref.abs().max()) > 0.5           # the comparison is not vacuous
    # the library evaluates the rotary angles in float32, hence 1e-5 rather than 1e-10
    assert float((out - ref).abs().max()) < 1e-5


# ---- closed forms ---------------------------------------------------------------------------------
def test_rope_closed_forms():
    g = torch.Generator().manual_seed(7)
    x = torch.randn(4, 3, 8, generator=g, dtype=F64)
    assert torch.equal(oracle.rope(x, torch.zeros(4, dtype=torch.long), 10000.0), x)   # position 0
    # hd = 2: a plane rotation by `pos` radians
    y = oracle.rope(torch.tensor([[[1.0, 0.0]]], dtype=F64), torch.tensor([3]), 123.0)
    assert torch.allclose(y, torch.tensor([[[math.cos(3.0), math.sin(3.0)]]], dtype=F64), atol=1e-15)
    # complex form: (x_i + i x_{i+hd/2}) * exp(i p theta^(-2i/hd))
    p = torch.tensor([0, 1, 5, 11])
    r = oracle.rope(x, p, 500.0)
    z = torch.complex(x[..., :4], x[..., 4:])
    ang = p.double()[:, None] * 500.0 ** (-2.0 * torch.arange(4, dtype=F64) / 8)
    zr = z * torch.polar(torch.ones_like(ang), ang)[:, None, :]
    assert torch.allclose(r, torch.cat([zr.real, zr.imag], -1), atol=1e-13)
    # relative-position property of the inner product
    q, k = x[0:1], x[1:2]
    a = (oracle.rope(q, torch.tensor([9]), 500.0) * oracle.rope(k, torch.tensor([4]), 500.0)).sum(-1)
    b = (oracle.rope(q, torch.tensor([25]), 500.0) * oracle.rope(k, torch.tensor([20]), 500.0)).sum(-1)
    assert torch.allclose(a, b, atol=1e-12)


def test_attention_degenerate_cases():
    g = torch.Generator().manual_seed(8)
    q = torch.randn(1, 2, 8, generator=g, dtype=F64)
    k = torch.randn(1, 2, 8, generator=g, dtype=F64)
    v = torch.randn(1, 2, 8, generator=g, dtype=F64)
    z = torch.zeros(1, dtype=torch.long)
    assert torch.allclose(oracle.attention(q, k, v, z, z), v, atol=1e-15)       # one key: output = v
    kk = k.expand(5, 2, 8).contiguous()
    vv = torch.randn(5, 2, 8, generator=g, dtype=F64)
    out = oracle.attention(q, kk, vv, torch.tensor([4]), torch.arange(5))
    assert torch.allclose(out[0], vv.mean(0), atol=1e-14)                       # equal keys: mean of v
    out = oracle.attention(q, kk, vv, torch.tensor([2]), torch.arange(5))       # causal cut at 2
    assert torch.allclose(out[0], vv[:3].mean(0), atol=1e-14)


def test_position_shift_invariance():
    s = _small_shape()
    m = oracle.OracleModel(s, _rand_weights(s, seed=9))
    toks = list(range(40, 52))
    a, b = m.forward_full(toks), m.forward_full(toks, pos_offset=37)
    assert torch.allclose(a, b, rtol=0, atol=1e-9)


# ---- invariants the paper states ------------------------------------------------------------------
def test_incremental_equals_full_recompute():
    s = _small_shape()
    m = oracle.OracleModel(s, _rand_weights(s, seed=10))
    toks = [int(x) for x in torch.randint(0, s.vocab, (21,), generator=torch.Generator().manual_seed(11))]
    full = m.forward_full(toks)
    cache = m.new_cache()
    rows = []
    for lo, hi in [(0, 7), (7, 8), (8, 16), (16, 21)]:
        rows.append(m.forward_chunk(toks[lo:hi], cache))
    assert torch.allclose(torch.cat(rows), full, rtol=0, atol=1e-10)
    assert cache.length == 21


def test_batched_layer_equals_one_sequence_at_a_time():
    """The layer over several sequences at once (what a batched verify step computes) is each sequence's own
    forward: rows of different sequences never meet.  Checked against separate full recomputes of three sequences
    of different lengths, split into a cached part and a chunk at different places."""
    s = _small_shape()
    m = oracle.OracleModel(s, _rand_weights(s, seed=12))
    g = torch.Generator().manual_seed(13)
    seqs = [[int(x) for x in torch.randint(0, s.vocab, (n,), generator=g)] for n in (19, 7, 30)]
    cuts = [11, 0, 29]                                        # cached tokens per sequence (one empty cache)
    caches = [m.new_cache() for _ in seqs]
    for toks, cut, c in zip(seqs, cuts, caches):
        if cut:
            m.forward_chunk(toks[:cut], c)
    xs = [m.w["embed"][torch.tensor(toks[cut:])].to(F64) for toks, cut in zip(seqs, cuts)]
    poss = [torch.arange(cut, len(toks)) for toks, cut in zip(seqs, cuts)]
    for l in range(s.n_layers):
        xs, _, _ = m._layer_multi(l, xs, poss, [c.k[l] for c in caches], [c.v[l] for c in caches],
                                  [torch.arange(cut) for cut in cuts])
    for toks, cut, x in zip(seqs, cuts, xs):
        want = m.forward_full(toks)[cut:]
        assert torch.allclose(m._head(x), want, rtol=0, atol=1e-10)


def test_verify_special_cases(tiny):
    s, w = tiny
    m = oracle.OracleModel(s, w)
    prompt = synth.make_context(s.vocab, 32)
    cache, pending = oracle.prefill(m, prompt)
    # ground truth continuation by vanilla greedy
    c2, p2, truth = cache.clone(), pending, []
    for _ in range(8):
        p2 = m.greedy_next(p2, c2)
        truth.append(p2)
    # k = 1 is one vanilla step
    r = m.verify(pending, [], cache.clone())
    assert r["accept_len"] == 0 and r["emitted"] == [truth[0]]
    # all-correct draft: everything accepted plus the bonus token
    c = cache.clone()
    r = m.verify(pending, truth[:7], c)
    assert r["accept_len"] == 7 and r["emitted"] == truth[:8] and c.length == cache.length + 8
    # corrupted at index p: exactly p accepted, emitted = truth[:p+1]
    for p in (0, 3, 6):
        bad = list(truth[:7])
        bad[p] = (bad[p] + 1) % s.vocab
        c = cache.clone()
        r = m.verify(pending, bad, c)
        assert r["accept_len"] == p and r["emitted"] == truth[:p + 1]
        assert c.length == cache.length + p + 1


def test_losslessness_and_mat(tiny):
    """Speculative output == vanilla greedy output, token for token; with empty drafts the mean
    number of tokens per step is exactly 1.00 (Table 3's vanilla row)."""
    s, w = tiny
    m = oracle.OracleModel(s, w)
    schema = synth.make_schema(s.vocab, 8)
    prompt = synth.make_context(s.vocab, 48)
    yv = oracle.vanilla_greedy(m, schema, prompt, eos=2, max_new_tokens=20)
    # a store that contains the model's own output: drafts get accepted
    store = oracle.Datastore(len(schema.tools))
    for tid, toks in synth.make_datastore(schema, 16):
        store.add(toks, tid)
    store.add(yv, 0)
    tr = []
    ys = oracle.speculative_decode(m, schema, store, prompt, eos=2, max_new_tokens=20, k_max=8, trace=tr)
    assert ys == yv
    assert len(tr) < len(yv) and any(t["accept_len"] > 0 for t in tr)
    tr = []
    ys = oracle.speculative_decode(m, schema, oracle.Datastore(8), prompt, eos=2,
                                   max_new_tokens=12, k_max=1, trace=tr)
    assert ys == yv[:12]
    assert sum(t["accept_len"] + 1 for t in tr) / len(tr) == 1.00


def test_argmax_ties_lowest_id():
    row = torch.tensor([[0.0, 3.0, 1.0, 3.0, 3.0]], dtype=F64)
    assert oracle.argmax_lowest(row) == [1]


def test_weight_blob_statistics():
    s = synth.SHAPES["tiny"]
    w = synth.make_weights(s)
    x = torch.cat([w[k].double().flatten() for k in w if w[k].dim() == 2])
    n = x.numel()
    assert abs(float(x.mean())) < 3 * 0.02 / math.sqrt(n)
    assert abs(float(x.std()) - 0.02) < 3 * 0.02 / math.sqrt(2 * n) + 0.02 * 2 ** -9
    assert all(bool((w[k] == 1).all()) for k in w if w[k].dim() == 1)
    w2 = synth.make_weights(s)
    assert all(torch.equal(w[k], w2[k]) for k in w)
