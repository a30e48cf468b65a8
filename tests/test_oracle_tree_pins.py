"""Pins for the tree-verification oracle (Appendix A.1, Algorithm 1's PackDraftsAsTree / Verification /
SelectLongestAcceptedPrefix): every test checks it against something other than itself -- the linear
step it generalises, a brute-force chain forward per node, vanilla greedy decoding, hand-built trees."""
import numpy as np
import torch

import oracle
import synth
from oracle.transformer import F64
from test_oracle_pins import _small_shape, _rand_weights


def _model(seed=3, **kw):
    shape = _small_shape(**kw)
    return shape, oracle.OracleModel(shape, _rand_weights(shape, seed=seed))


def _prefilled(om, n, seed=0):
    g = np.random.Generator(np.random.Philox(key=[seed, 77]))
    prompt = [int(t) for t in g.integers(8, om.s.vocab, size=n + 1)]
    return oracle.prefill(om, prompt)          # cache with n tokens, last one pending


def _random_tree(g, k, vocab):
    parents = [-1] + [int(g.integers(0, j)) for j in range(1, k)]
    tokens = [int(t) for t in g.integers(8, vocab, size=k - 1)]
    return tokens, parents


def test_chain_tree_is_the_linear_step_bitwise():
    shape, om = _model()
    cache, pending = _prefilled(om, 19)
    g = np.random.Generator(np.random.Philox(key=[5, 1]))
    draft = [int(t) for t in g.integers(8, shape.vocab, size=6)]
    c1, c2 = cache.clone(), cache.clone()
    lin = om.verify(pending, draft, c1, want_logits=True)
    tree = oracle.verify_tree(om, pending, draft, [-1, 0, 1, 2, 3, 4, 5], c2, want_logits=True)
    assert torch.equal(lin["logits"], tree["logits"])
    assert lin["accept_len"] == tree["accept_len"] and lin["emitted"] == tree["emitted"]
    assert tree["path"] == list(range(lin["accept_len"] + 1))
    for l in range(shape.n_layers):
        assert torch.equal(c1.k[l], c2.k[l]) and torch.equal(c1.v[l], c2.v[l])


def test_every_node_equals_a_chain_forward_of_its_root_path():
    """Brute force: a node's logits are those of the last row of an ordinary chunk forward over the
    tokens on its root path, whatever else is in the tree."""
    shape, om = _model(seed=4)
    cache, pending = _prefilled(om, 11, seed=2)
    g = np.random.Generator(np.random.Philox(key=[5, 2]))
    tokens, parents = _random_tree(g, 12, shape.vocab)
    z = [pending] + tokens
    logits, k_new, v_new = oracle.forward_tree(om, z, parents, cache)
    for j in range(len(z)):
        path, u = [], j
        while u >= 0:
            path.append(u)
            u = parents[u]
        path.reverse()
        c = cache.clone()
        ref = om.forward_chunk([z[i] for i in path], c)
        assert torch.allclose(logits[j], ref[-1], rtol=0, atol=1e-9), f"node {j}"
        for l in range(shape.n_layers):                      # and its K/V rows are the chain's last rows
            assert torch.allclose(k_new[l][j], c.k[l][-1], rtol=0, atol=1e-10)
            assert torch.allclose(v_new[l][j], c.v[l][-1], rtol=0, atol=1e-10)


def test_siblings_do_not_see_each_other():
    shape, om = _model(seed=5)
    cache, pending = _prefilled(om, 7, seed=3)
    #        0
    #      /   \
    #     1     3
    #     |     |
    #     2     4
    parents = [-1, 0, 1, 0, 3]
    a = [pending, 100, 101, 200, 201]
    b = [pending, 100, 101, 300, 301]          # other branch changed
    la, _, _ = oracle.forward_tree(om, a, parents, cache)
    lb, _, _ = oracle.forward_tree(om, b, parents, cache)
    assert torch.equal(la[:3], lb[:3])
    assert not torch.allclose(la[3:], lb[3:])


def test_ancestor_mask_and_depths_by_hand():
    parents = [-1, 0, 0, 1, 3, 2]
    assert oracle.node_depths(parents) == [0, 1, 1, 2, 3, 2]
    m = oracle.ancestor_mask(parents).int().tolist()
    assert m == [[1, 0, 0, 0, 0, 0],
                 [1, 1, 0, 0, 0, 0],
                 [1, 0, 1, 0, 0, 0],
                 [1, 1, 0, 1, 0, 0],
                 [1, 1, 0, 1, 1, 0],
                 [1, 0, 1, 0, 0, 1]]


def test_accepted_path_walk_by_hand():
    z = [9, 5, 6, 7, 6, 8]
    parents = [-1, 0, 0, 1, 2, 4]
    # model tokens per node: root says 6 -> node 2; node 2 says 6 -> node 4; node 4 says 1 -> stop
    assert oracle.accepted_path(z, parents, [6, 0, 6, 0, 1, 0]) == [0, 2, 4]
    assert oracle.accepted_path(z, parents, [4, 0, 0, 0, 0, 0]) == [0]                 # nothing matches
    assert oracle.accepted_path(z, parents, [5, 7, 0, 3, 0, 0]) == [0, 1, 3]
    # duplicate sibling tokens (malformed trie): the lowest-numbered child wins
    assert oracle.accepted_path([9, 5, 5], [-1, 0, 0], [5, 0, 0]) == [0, 1]


def test_pack_candidates_builds_a_trie_in_creation_order():
    toks, par = oracle.pack_candidates([[1, 2, 3], [1, 2, 4, 5], [7], [1, 9]], max_nodes=64)
    assert toks == [1, 2, 3, 4, 5, 7, 9]
    assert par == [-1, 0, 1, 2, 2, 4, 0, 1]
    toks, par = oracle.pack_candidates([[1, 2, 3], [1, 2, 4, 5]], max_nodes=5)           # budget: root + 4
    assert toks == [1, 2, 3, 4] and par == [-1, 0, 1, 2, 2]
    assert oracle.pack_candidates([], 8) == ([], [-1])


def test_tree_decoding_equals_vanilla_greedy_and_keeps_the_right_cache():
    """Losslessness (Section 5.2, Table 5) with trees: whatever the candidates are, the emitted
    stream is the greedy stream, and the compacted cache equals the cache of plain incremental
    decoding over the same tokens."""
    shape, om = _model(seed=6)
    cache0, pending0 = _prefilled(om, 9, seed=4)
    # vanilla stream
    c, p, ref = cache0.clone(), pending0, []
    for _ in range(24):
        p = om.greedy_next(p, c)
        ref.append(p)
    g = np.random.Generator(np.random.Philox(key=[5, 3]))
    c, p, out, steps = cache0.clone(), pending0, [], 0
    while len(out) < 24:
        done = len(out)
        truth = ref[done:done + int(g.integers(0, 6))]             # a correct candidate of random length
        wrong1 = truth[:max(0, len(truth) - 2)] + [int(t) for t in g.integers(8, shape.vocab, size=3)]
        wrong2 = [int(t) for t in g.integers(8, shape.vocab, size=4)]
        cands = [wrong2, truth, wrong1]
        toks, par = oracle.pack_candidates(cands, max_nodes=16)
        res = oracle.verify_tree(om, p, toks, par, c)
        assert res["accept_len"] >= len(truth)                     # the greedy continuation is always accepted
        out += res["emitted"]
        p = res["emitted"][-1]
        steps += 1
    assert out[:24] == ref
    assert steps < 24                                              # some drafts were accepted
    # the cache now holds pending0 + out[:-1]; compare with plain incremental decoding over them
    plain = cache0.clone()
    om.forward_chunk([pending0] + out[:-1], plain)
    assert plain.length == c.length
    for l in range(shape.n_layers):
        assert torch.allclose(plain.k[l], c.k[l], rtol=0, atol=1e-9)
        assert torch.allclose(plain.v[l], c.v[l], rtol=0, atol=1e-9)


def test_sibling_order_does_not_change_the_result():
    shape, om = _model(seed=7)
    cache, pending = _prefilled(om, 10, seed=5)
    t0 = om.greedy_next(pending, cache.clone())
    c = cache.clone()
    om.forward_chunk([pending], c)
    t1 = om.greedy_next(t0, c)
    cands_a = [[t0, t1, 50], [60, 61], [t0, 70]]
    cands_b = [[60, 61], [t0, 70], [t0, t1, 50]]
    ra = oracle.verify_tree(om, pending, *oracle.pack_candidates(cands_a, 32), cache.clone())
    rb = oracle.verify_tree(om, pending, *oracle.pack_candidates(cands_b, 32), cache.clone())
    assert ra["emitted"] == rb["emitted"] and ra["accept_len"] == rb["accept_len"] >= 2
