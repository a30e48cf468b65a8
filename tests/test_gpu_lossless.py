"""Losslessness on the GPU path (paper Section 5.2, Table 5: the speculative output is the target model's own output).

The oracle pins this property on the CPU (tests/test_oracle_pins.py); here it is required of the CUDA path itself, bit for
bit: a row's logits must not depend on how many other rows are verified in the same step.  Then the argmax of row j of
a chunk IS the token vanilla decoding would produce after the same prefix, and the decode loop of Algorithm 1 emits the
vanilla sequence whatever the drafts are.

  * row invariance: the first rows of a k = 32 step equal, bitwise, the rows of k = 1 / k = 8 steps over the same
    prefix (chains), and the root and first branch of a draft tree equal the chain's rows;
  * the loop: 512 tokens by k = 1 steps, then the same context again through ts_draft -> ts_verify -> ts_commit with
    drafts retrieved from that output and corrupted at seeded places: identical ids, no tolerance.
"""
import numpy as np
import pytest
import torch

import synth
import paper_2604_13519_b200 as ts
from synth.toolcalls import planted_accept_lengths

pytestmark = pytest.mark.gpu

PATHS = [pytest.param(1, id="separate"), pytest.param(2, id="fused")]


def _model(shape, k_max, max_ctx, path, gain_seed=None):
    w = synth.make_weights(shape, gain_seed=gain_seed)
    gm = ts.Model(shape, max_pages=(max_ctx + 15) // 16 + 4, max_batch=1, k_max=k_max, max_rows=k_max, max_ctx=max_ctx,
                  act_split=True, path=path)
    gm.load_weights(w)
    return gm


def _context(shape, gm, length, stream=0):
    K, V = synth.make_synthetic_kv(shape, length, stream=stream)
    s = ts.Session(gm, None, None)
    for l in range(shape.n_layers):
        s.import_kv(l, K[l], V[l])
    s.set_cache(length, synth.Vocab(shape.vocab).tool_call)
    return s


def _draft(vocab, n, seed):
    g = torch.Generator().manual_seed(seed)
    return [int(x) for x in torch.randint(64, vocab, (n,), generator=g)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,ctx", [("8b-2l", 700), ("8b-2l", 2048), ("1b-2l", 1000), ("tiny", 37), ("8b-2l", 0)])
def test_rows_do_not_depend_on_chunk_length(name, ctx, path):
    shape = synth.SHAPES[name]
    gm = _model(shape, 32, ctx + 64, path, gain_seed=7)
    s = _context(shape, gm, ctx)
    d = _draft(shape.vocab, 31, 11)
    ts.ts_verify(gm, [s], [d])
    full = gm.read_logits(0, 32).copy()
    for k in (1, 2, 8, 17):
        r = ts.ts_verify(gm, [s], [d[:k - 1]])[0]
        assert r.k == k
        got = gm.read_logits(0, k)
        assert np.array_equal(got, full[:k]), f"{name} ctx={ctx} path={path}: rows of a k={k} step differ from the k=32 step"
    gm.close()


@pytest.mark.parametrize("name,ctx", [("8b-2l", 700), ("1b-2l", 130)])
def test_tree_rows_equal_chain_rows(name, ctx):
    """A draft tree: the root and the nodes of its first branch (nodes 1..8, a chain) carry the logits of the same ids
    verified as a plain chain; the other branches only add masked columns."""
    shape = synth.SHAPES[name]
    gm = _model(shape, 32, ctx + 64, 1, gain_seed=7)
    s = _context(shape, gm, ctx)
    d = _draft(shape.vocab, 31, 13)
    ts.ts_verify(gm, [s], [d[:8]])
    chain = gm.read_logits(0, 9).copy()
    # branch A: nodes 1..8 under the root; branch B: 12 nodes under the root; branch C: 11 nodes under node 3
    parents = [0] + list(range(1, 8)) + [0] + list(range(9, 20)) + [3] + list(range(21, 31))
    assert len(parents) == 31
    ts.ts_verify_tree(gm, [s], [d], [parents])
    tree = gm.read_logits(0, 9)
    assert np.array_equal(tree, chain)
    gm.close()


def test_speculative_output_equals_vanilla_output():
    """512 tokens on the 8B layer shape (2 layers), 700-token context: vanilla decoding, then the loop of Algorithm 1
    with retrieval drafts of up to 31 ids taken from that output and corrupted at seeded indices."""
    shape = synth.SHAPES["8b-2l"]
    n_tokens, ctx = 512, 700
    gm = _model(shape, 32, ctx + n_tokens + 96, 1, gain_seed=7)
    store = ts.Datastore(1)
    K, V = synth.make_synthetic_kv(shape, ctx)
    s = ts.Session(gm, None, store)
    for l in range(shape.n_layers):
        s.import_kv(l, K[l], V[l])
    pending = synth.Vocab(shape.vocab).tool_call
    s.set_cache(ctx, pending)
    for _ in range(n_tokens):
        ts.ts_commit(s, ts.ts_verify(gm, [s], [[]])[0])
    vanilla = s.output()
    assert len(vanilla) == n_tokens
    store.add(vanilla, 0)
    planted = planted_accept_lengths(n_tokens)
    s.restart(ctx, pending)
    steps, accepted = 0, []
    while s.state().n_output < n_tokens:
        d, _src = ts.ts_draft(s, min(31, n_tokens - s.state().n_output))
        if planted[steps] < len(d):
            d[planted[steps]] = (d[planted[steps]] + 1) % shape.vocab
        r = ts.ts_verify(gm, [s], [d])[0]
        ts.ts_commit(s, r)
        accepted.append(r.accept_len)
        steps += 1
    out = s.output()
    assert out[:n_tokens] == vanilla, "speculative decoding left the vanilla trajectory"
    assert steps < n_tokens // 3 and max(accepted) >= 16        # the drafts were really accepted, in long spans too
    gm.close()
