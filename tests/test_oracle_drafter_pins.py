"""Pins for the drafter oracle: printed constants, grammar validity checked by an independent
recursive-descent validator, brute force over all (L, candidate, position) triples, and the
priority of retrieval over schema drafting (Algorithm 1)."""
import os
import random

import oracle
import synth
from oracle.drafter import Q_O, Q_T, Q_P, Q_V, Q_DONE

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


def test_printed_constants():
    g = _gold()
    assert tuple(int(x) for x in g["suffix_lengths"].split()) == oracle.SUFFIX_LENGTHS
    assert int(g["continuation_lengths"].split()[0]) == oracle.DEFAULT_N_CAP
    assert g["fsm_states"].split() == [Q_T, Q_P, Q_V, Q_O]


def _schema(seed=1, n_tools=12):
    return synth.make_schema(4096, n_tools, seed=seed)


def _store(schema, n=64, seed=1):
    st = oracle.Datastore(len(schema.tools))
    inv = synth.make_datastore(schema, n, seed=seed)
    for tid, toks in inv:
        st.add(toks, tid)
    return st, inv


def test_fsm_walks_every_invocation_and_drafts_are_valid():
    schema = _schema()
    st, inv = _store(schema)
    v = schema.vocab
    for tid, toks in inv[:40]:
        d = oracle.Drafter(schema, oracle.Datastore(len(schema.tools)))   # no retrieval
        d.feed_prompt([77, 99, v.tool_call])
        assert d.fsm.kind == Q_T
        for i, t in enumerate(toks):
            draft = d.fsm.draft(d.guess_tool)
            # every schema draft extends the output to a prefix of some valid invocation
            assert oracle.validate_prefix(schema, toks[:i] + draft), (tid, i, draft)
            # once the tool is known the filling is deterministic: it must equal the real continuation
            if d.fsm.kind in (Q_P,) or (d.fsm.kind == Q_T and d.fsm.stage == "mid") or \
                    (d.fsm.kind == Q_V and d.fsm.stage in ("nxt", "end")):
                assert draft and toks[i:i + len(draft)] == draft
            if d.fsm.kind == Q_V and d.fsm.stage == "val":
                assert draft == []
            d.commit([t], v.eos, 10 ** 6)
        assert d.fsm.kind == Q_DONE and d.fsm.tool == tid
        assert d.finished(v.eos, 10 ** 6)


def test_fsm_delimiters_and_off_schema():
    schema = _schema()
    v = schema.vocab
    tool = next(t for t in schema.tools if len(t.keys) >= 2)
    tid = schema.tools.index(tool)
    f = oracle.SchemaFsm(schema)
    for t in [v.tool_call] + list(v.pfx) + tool.name + list(v.mid):
        f.step(t)
    assert (f.kind, f.tool, f.key) == (Q_P, tid, 0)
    for t in tool.keys[0] + list(v.kvsep):
        f.step(t)
    assert f.kind == Q_V
    f.step(v.value_lo + 5)
    assert f.kind == Q_V and f.stage == "val"
    for t in v.nxt:                        # the '", "' delimiter returns to q_p for the next key
        f.step(t)
    assert (f.kind, f.key) == (Q_P, 1)
    for t in tool.keys[1] + list(v.kvsep) + [v.value_lo + 9] + list(v.end):   # '"}}' completes
        f.step(t)
    assert f.kind == Q_DONE
    # off-schema id in a structural state drops to q_o; <tool_call> re-enters q_t
    f = oracle.SchemaFsm(schema)
    for t in [v.tool_call, v.pfx[0], 999]:
        f.step(t)
    assert f.kind == Q_O
    f.step(v.tool_call)
    assert f.kind == Q_T and f.draft(lambda p: 0)[:3] == list(v.pfx)


def test_tool_guess_rules():
    schema = _schema(seed=3, n_tools=16)
    st, inv = _store(schema, n=80, seed=3)
    d = oracle.Drafter(schema, st)
    # no rank list: most frequent compatible tool, lowest id on ties
    comp = list(range(len(schema.tools)))
    best = max(comp, key=lambda t: (st.freq[t], -t))
    assert d.guess_tool([]) == best
    # shared first token: the guess stays compatible with the prefix
    for t, tool in enumerate(schema.tools):
        g = d.guess_tool(tool.name[:1])
        assert schema.tools[g].name[:1] == tool.name[:1]
        assert d.guess_tool(tool.name) in d.fsm.compatible_tools(tool.name)
    # with a rank list the first ranked candidate's tool wins
    ranks = [5, 9, 2]
    d2 = oracle.Drafter(schema, st, ranks=ranks)
    assert d2.guess_tool([]) == st.tool_of[5]
    # empty datastore: lowest compatible id
    d3 = oracle.Drafter(schema, oracle.Datastore(len(schema.tools)))
    assert d3.guess_tool([]) == 0


def _brute_force(y, entries, order, n):
    hits = []
    for L in (5, 6, 7):
        if len(y) < L:
            continue
        for rank, c in enumerate(order):
            e = entries[c]
            for m in range(L, len(e)):
                if e[m - L:m] == list(y[-L:]):
                    hits.append((-L, rank, m, c))
    if not hits:
        return [], None
    negL, rank, m, c = min(hits)
    return entries[c][m:m + n], (-negL, c, m)


def test_suffix_match_equals_brute_force():
    rnd = random.Random(5)
    for trial in range(200):
        alphabet = rnd.choice([2, 3, 5])
        n_e = rnd.randint(1, 6)
        st = oracle.Datastore(1)
        for _ in range(n_e):
            st.add([rnd.randrange(alphabet) for _ in range(rnd.randint(1, 30))], 0)
        y = [rnd.randrange(alphabet) for _ in range(rnd.randint(0, 12))]
        ranks = None if trial % 2 else rnd.sample(range(n_e), rnd.randint(1, n_e))
        n_cap, max_draft = rnd.choice([1, 4, 32]), rnd.choice([1, 7, 63])
        got, where = oracle.suffix_match(y, st, ranks, n_cap, max_draft)
        order = list(range(n_e)) if ranks is None else ranks
        ref, ref_where = _brute_force(y, st.entries, order, min(n_cap, max_draft))
        assert got == ref
        if ref_where is not None:
            assert where == ref_where


def test_suffix_priorities():
    st = oracle.Datastore(1)
    st.add([1, 2, 3, 4, 5, 6, 7, 100, 101], 0)            # matches with L = 7
    st.add([9, 3, 4, 5, 6, 7, 200, 201], 0)                  # matches only with L = 5
    y = [0, 1, 2, 3, 4, 5, 6, 7]
    assert oracle.suffix_match(y, st, None, 32, 63)[0] == [100, 101]
    assert oracle.suffix_match(y, st, [1, 0], 32, 63)[0] == [100, 101]      # longer L beats rank
    assert oracle.suffix_match(y[3:], st, [1, 0], 32, 63)[0] == [200, 201]  # same L: rank order
    assert oracle.suffix_match(y[4:], st, None, 32, 63)[0] == []            # shorter than 5: no match
    st2 = oracle.Datastore(1)
    st2.add([3, 4, 5, 6, 7], 0)                               # match at the very end: no continuation
    assert oracle.suffix_match(y, st2, None, 32, 63)[0] == []
    long = oracle.Datastore(1)
    long.add(list(range(10, 17)) + list(range(100, 200)), 0)
    assert len(oracle.suffix_match(list(range(10, 17)), long, None, 32, 63)[0]) == 32
    assert len(oracle.suffix_match(list(range(10, 17)), long, None, 64, 63)[0]) == 63


def test_retrieval_has_priority_over_schema():
    schema = _schema()
    st, inv = _store(schema)
    tid, toks = inv[0]
    v = schema.vocab
    d = oracle.Drafter(schema, st)
    d.feed_prompt([v.tool_call])
    draft, src = d.draft(16)
    assert src == 1 and draft[:3] == list(v.pfx)            # |y| < 5: schema draft
    d.commit(toks[:9], v.eos, 10 ** 6)
    draft, src = d.draft(16)
    assert src == 2                                          # a 7-gram of history matches
    hit = next(e for e in st.entries if any(e[m - 7:m] == toks[2:9] for m in range(7, len(e))))
    m = next(m for m in range(7, len(hit)) if hit[m - 7:m] == toks[2:9])
    assert draft == hit[m:m + 16]
    assert d.draft(0) == ([], 0)


def test_commit_stops_at_finish():
    schema = _schema()
    st, inv = _store(schema)
    tid, toks = inv[3]
    v = schema.vocab
    d = oracle.Drafter(schema, st)
    d.feed_prompt([v.tool_call])
    n, fin = d.commit(toks + [555, 666], v.eos, 10 ** 6)
    assert fin and n == len(toks) and d.y == toks
    d = oracle.Drafter(schema, st)
    n, fin = d.commit([70, 71, v.eos, 72], v.eos, 10 ** 6)
    assert fin and n == 3
    d = oracle.Drafter(schema, st)
    n, fin = d.commit([70, 71, 72, 73], v.eos, 3)
    assert fin and n == 3


def test_validator_rejects_bad_sequences():
    schema = _schema()
    st, inv = _store(schema)
    tid, toks = inv[0]
    assert oracle.validate_prefix(schema, toks)
    assert oracle.validate_prefix(schema, toks[:5])
    bad = list(toks)
    bad[1] = 999
    assert not oracle.validate_prefix(schema, bad)
    assert not oracle.validate_prefix(schema, toks + [70])
    tool = schema.tools[tid]
    if len(tool.keys) >= 2:     # keys out of order
        v = schema.vocab
        swapped = list(v.pfx) + tool.name + list(v.mid) + tool.keys[1] + list(v.kvsep)
        assert tool.keys[0] == tool.keys[1] or not oracle.validate_prefix(schema, swapped)


# ---- candidate sets and PackDraftsAsTree (Algorithm 1; Appendix B.2's continuation lengths) --------------
def test_continuation_lengths_are_the_printed_ones():
    g = _gold()
    assert tuple(int(x) for x in g["continuation_lengths"].split()) == (oracle.DEFAULT_N_CAP,) + oracle.drafter.LATER_CAPS


def _brute_force_hits(y, entries, order, caps, max_draft):
    hits = []
    for L in (5, 6, 7):
        if len(y) < L:
            continue
        for rank, c in enumerate(order):
            e = entries[c]
            for m in range(L, len(e)):
                if e[m - L:m] == list(y[-L:]):
                    hits.append((-L, rank, m, c))
    out, seen = [], set()
    for negL, rank, m, c in sorted(hits):
        if (c, m) in seen:
            continue
        seen.add((c, m))
        out.append(entries[c][m:m + min(caps[len(out)], max_draft)])
        if len(out) == len(caps):
            break
    return out


def test_suffix_matches_equal_brute_force_and_start_with_the_chain_draft():
    rnd = random.Random(11)
    nonempty = 0
    for trial in range(300):
        alphabet = rnd.choice([2, 3, 5])
        n_e = rnd.randint(1, 6)
        st = oracle.Datastore(1)
        for _ in range(n_e):
            st.add([rnd.randrange(alphabet) for _ in range(rnd.randint(1, 40))], 0)
        y = [rnd.randrange(alphabet) for _ in range(rnd.randint(0, 12))]
        ranks = None if trial % 2 else rnd.sample(range(n_e), rnd.randint(1, n_e))
        caps = (rnd.choice([1, 4, 32]), 16, 8, 8)
        max_draft = rnd.choice([1, 7, 63])
        got = oracle.suffix_matches(y, st, ranks, caps, max_draft)
        order = list(range(n_e)) if ranks is None else ranks
        assert got == _brute_force_hits(y, st.entries, order, caps, max_draft)
        first, _ = oracle.suffix_match(y, st, ranks, caps[0], max_draft)
        assert (got[0] if got else []) == first
        nonempty += len(got) > 1
    assert nonempty > 20          # several hits do occur in this sweep


def _leaf_paths(tokens, parents):
    kids = {}
    for j in range(1, len(parents)):
        kids.setdefault(parents[j], []).append(j)
    out = []

    def walk(u, acc):
        if u not in kids:
            out.append(acc)
        for c in kids.get(u, []):
            walk(c, acc + [tokens[c - 1]])
    walk(0, [])
    return out


def test_tool_name_candidates_are_valid_and_cover_the_guess():
    schema = _schema(seed=3, n_tools=12)
    st, inv = _store(schema, seed=3)
    v = schema.vocab
    for tid, toks in inv[:30]:
        d = oracle.Drafter(schema, oracle.Datastore(len(schema.tools)))       # no retrieval
        d.feed_prompt([77, v.tool_call])
        for i, t in enumerate(toks):
            cands, src = d.draft_candidates(63)
            chain, csrc = d.draft(63)
            assert (cands[0] if cands else []) == chain and src == csrc       # first candidate = chain draft
            toks_t, par_t, _ = d.draft_tree(64)
            for leaf in _leaf_paths(toks_t, par_t):
                assert oracle.validate_prefix(schema, toks[:i] + leaf), (tid, i, leaf)
            if d.fsm.kind == Q_T and d.fsm.stage != "mid":
                # with the name open, the true tool is among the candidates whenever at most
                # MAX_TOOL_CANDIDATES tools are compatible, and then its whole scaffold is a root path
                prefix = [] if d.fsm.stage == "pfx" else d.fsm.name_prefix
                comp = d.fsm.compatible_tools(prefix)
                assert len(cands) == min(len(comp), oracle.drafter.MAX_TOOL_CANDIDATES)
                if len(comp) <= oracle.drafter.MAX_TOOL_CANDIDATES:
                    truth = d.fsm.draft(lambda _p: tid)
                    assert truth in cands and toks[i:i + len(truth)] == truth
            else:
                assert len(cands) <= 1
            d.commit([t], v.eos, 10 ** 6)


def test_tree_loop_equals_vanilla_greedy_on_a_tiny_model():
    """Algorithm 1 with candidate trees preserves the model's output (Section 5.2, Table 5)."""
    import torch  # noqa: F401
    from test_oracle_pins import _small_shape, _rand_weights
    shape = _small_shape(vocab=4096)
    om = oracle.OracleModel(shape, _rand_weights(shape, seed=9))
    schema = _schema(seed=4, n_tools=8)
    v = schema.vocab
    st, inv = _store(schema, n=32, seed=4)
    prompt = synth.make_context(4096, 24, seed=4)
    ref = oracle.vanilla_greedy(om, schema, prompt, v.eos, 40)
    # self-history: the model's own output, intact and with planted errors, among the historical invocations
    bad = list(ref)
    for p in (8, 19, 30):
        bad[p] = (bad[p] + 1) % 4096
    for e in (bad, ref, ref[:15] + bad[15:]):
        st.add(e, -1)
    trace = []
    out = oracle.speculative_decode_tree(om, schema, st, prompt, v.eos, 40, max_nodes=24, trace=trace)
    assert out == ref
    assert len(trace) < len(ref)                                     # drafts were accepted
    assert any(len(set(t["parents"])) < len(t["parents"]) for t in trace)       # and some trees did branch


# ---- general speculative drafting for q_v / q_o: context match and recycled successors ----------------------
def test_context_match_equals_brute_force():
    rnd = random.Random(21)
    hits = 0
    for _ in range(300):
        alphabet = rnd.choice([2, 3, 6])
        ctx = [rnd.randrange(alphabet) for _ in range(rnd.randint(0, 40))]
        n = rnd.choice([1, 5, 32])
        best = None
        for L in (5, 6, 7):
            if len(ctx) <= L:
                continue
            for m in range(L, len(ctx)):
                if ctx[m - L:m] == ctx[-L:]:
                    key = (-L, m)
                    if best is None or key < best:
                        best = key
        want = [] if best is None else ctx[best[1]:best[1] + n]
        assert oracle.context_match(ctx, n) == want
        hits += bool(want)
    assert hits > 30
    assert oracle.context_match([1, 2, 3, 4, 5], 4) == []            # the suffix matching itself does not count


def test_recycled_tree_shape_and_lookup():
    class Every(dict):                                # a list for every token: 10 t + rank + 1
        def __contains__(self, t):
            return True

        def __getitem__(self, t):
            return [10 * t + r + 1 for r in range(oracle.TOPK)]
    table = Every()
    toks, par = oracle.recycled_tree(1, table, 64)
    assert len(toks) == 17 and par[0] == -1
    # every node carries the successor of its parent's token at the template's rank, parents come first
    z = [1] + toks
    kids = {}
    for j in range(1, len(z)):
        assert 0 <= par[j] < j
        r = kids.setdefault(par[j], 0)
        assert z[j] == table[z[par[j]]][r]           # children of a node appear in rank order 0, 1, 2, ...
        kids[par[j]] = r + 1
    assert kids[0] == 4 and sorted(kids.values(), reverse=True)[:4] == [4, 3, 2, 2]
    depth = oracle.node_depths(par)
    assert max(depth) == 5 and depth.count(1) == 4 and depth.count(2) == 7
    # the budget cuts in slot order; a token without a list prunes its subtree
    assert oracle.recycled_tree(1, table, 6)[1] == [-1, 0, 0, 0, 0, 1]
    class AllBut(Every):                              # the first child has no list: its whole subtree goes
        def __contains__(self, t):
            return t != table[1][0]
    toks2, par2 = oracle.recycled_tree(1, AllBut(), 64)
    assert len(toks2) == 17 - 8                       # slots 5, 6, 7, 12, 13, 14, 16, 17 hang below slot 1
    assert all(p != 1 for p in par2[1:])
    assert oracle.recycled_tree(7, {}, 64) == ([], [-1])


def test_topk_lowest_against_torch_and_ties():
    import torch
    g = torch.Generator().manual_seed(4)
    x = torch.randn(500, generator=g, dtype=torch.float64)
    assert oracle.topk_lowest(x, 8) == torch.topk(x, 8).indices.tolist()
    assert oracle.topk_lowest(torch.tensor([1.0, 3.0, 3.0, 0.0, 3.0]), 4) == [1, 2, 4, 0]


def test_general_sd_loop_is_lossless_and_uses_both_sources():
    from test_oracle_pins import _small_shape, _rand_weights
    shape = _small_shape(vocab=4096)
    om = oracle.OracleModel(shape, _rand_weights(shape, seed=12))
    schema = _schema(seed=5, n_tools=8)
    v = schema.vocab
    st = oracle.Datastore(len(schema.tools))          # empty: nothing to retrieve, q_o throughout
    prompt = synth.make_context(4096, 30, seed=5)[:-1] + [77]        # no tool call: the FSM stays in q_o
    ref = oracle.vanilla_greedy(om, schema, prompt, v.eos, 48)
    trace = []
    out = oracle.speculative_decode_tree(om, schema, st, prompt, v.eos, 48, max_nodes=20, trace=trace,
                                         general_sd=True)
    assert out == ref
    srcs = {t["source"] for t in trace}
    assert 4 in srcs                                   # recycled trees were drafted once lists existed
    assert trace[0]["source"] == 0                     # nothing to draft from at the very first step
