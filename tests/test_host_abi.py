"""CPU-only checks of the boundary: the library loads, exports every declared symbol, validates
arguments, and its host C++ drafter (FSM, datastore index, commit) is bit-exact with the oracle."""
import ctypes as C
import os
import random
import re

import pytest

import oracle
import synth
import paper_2604_13519_b200 as ts
from paper_2604_13519_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2604_13519_b200 import build
    build.build()


def test_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "toolspec.h")).read()
    declared = set(re.findall(r"^(?:ts_status|const char \*)\s*(ts_[a-z_0-9]+)\s*\(", hdr, re.M))
    assert {"ts_init_model", "ts_draft", "ts_verify", "ts_commit"} <= declared
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(B.EXPORTED)


def test_debug_library_builds_and_exports_the_same_symbols():
    """The debug build (every index a kernel takes from the step's inputs checked on the device) is the same library
    compiled with TS_DEBUG_BOUNDS: it must build and export every declared entry point."""
    from paper_2604_13519_b200 import build
    path = build.build(debug_bounds=True)
    assert path == B.DEBUG_LIB_PATH and os.path.exists(path)
    L = C.CDLL(path)
    for name in B.EXPORTED:
        assert hasattr(L, name), name
    assert B.STATUS[-9] == "TS_ERR_DEVICE_BOUNDS"
    hdr = open(os.path.join(ROOT, "include", "toolspec.h")).read()
    assert re.search(r"TS_ERR_DEVICE_BOUNDS\s*=\s*-9", hdr)


def test_buffer_sizes_and_argument_errors():
    c = B.ts_model_config()
    s = synth.SHAPES["8b"]
    for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "rope_theta", "rms_eps"):
        setattr(c, n, getattr(s, n))
    c.max_pages, c.max_batch, c.k_max, c.max_rows, c.max_ctx, c.act_split = 1024, 1, 32, 32, 16384, 1
    out = B.ts_buffer_sizes()
    assert B.lib().ts_query_buffer_sizes(C.byref(c), C.byref(out)) == 0
    w_expect = 2 * (s.n_params_matmul() + s.vocab * s.d_model)
    assert w_expect <= out.weights_bytes < w_expect * 1.001 + (1 << 20)
    assert out.kv_pool_bytes == 1024 * 16 * s.n_kv_heads * s.head_dim * 2 * 2 * s.n_layers
    c.head_dim = 96
    assert B.lib().ts_query_buffer_sizes(C.byref(c), C.byref(out)) == -1
    assert b"head_dim" in B.lib().ts_last_error()
    c.head_dim, c.k_max = 128, 65
    assert B.lib().ts_query_buffer_sizes(C.byref(c), C.byref(out)) == -1
    assert B.lib().ts_query_buffer_sizes(None, C.byref(out)) == -1
    # no device here (or no model): the verify entry point must fail, never fall back
    assert B.lib().ts_verify(None, None, 1, None, None, 0, None) == -1
    assert B.lib().ts_verify_replay(None) == -1


def _pair(schema, inv, n_cap=32, ranks=None, max_new=10 ** 6):
    st_o = oracle.Datastore(len(schema.tools))
    st_c = ts.Datastore(len(schema.tools))
    for tid, toks in inv:
        st_o.add(toks, tid)
        st_c.add(toks, tid)
    sc = ts.Schema(schema.vocab, schema.tools)
    d = oracle.Drafter(schema, st_o, n_cap=n_cap, ranks=ranks)
    s = ts.Session(None, sc, st_c, n_cap=n_cap, max_new_tokens=max_new)
    if ranks is not None:
        s.set_ranks(ranks)
    return d, s


KIND = {oracle.Q_O: 0, oracle.Q_T: 1, oracle.Q_P: 2, oracle.Q_V: 3, oracle.Q_DONE: 4}


@pytest.mark.parametrize("seed,n_tools,n_inv,ranks", [(1, 8, 64, None), (2, 32, 300, None), (3, 16, 100, [7, 3, 50, 9])])
def test_draft_and_commit_bit_exact_with_oracle(seed, n_tools, n_inv, ranks):
    schema = synth.make_schema(4096, n_tools, seed=seed)
    inv = synth.make_datastore(schema, n_inv, seed=seed)
    rnd = random.Random(seed)
    v = schema.vocab
    for trial in range(40):
        d, s = _pair(schema, inv, ranks=ranks, max_new=200)
        prompt = [rnd.randrange(64, 4096) for _ in range(5)] + [v.tool_call]
        d.feed_prompt(prompt)
        ts.ts_prefill(None, s, prompt)
        # script: a historical invocation, perturbed in places so that both drafters see misses,
        # off-schema ids and early stops
        tid, script = inv[rnd.randrange(len(inv))]
        script = list(script)
        for _ in range(rnd.randrange(0, 3)):
            script[rnd.randrange(len(script))] = rnd.randrange(64, 4096)
        script += [rnd.randrange(64, 4096) for _ in range(10)] + [v.eos]
        pos = 0
        while pos < len(script):
            md = rnd.choice([0, 1, 5, 31, 63])
            want, src = d.draft(md)
            got, gsrc = ts.ts_draft(s, md)
            assert (got, gsrc) == (want, src), (trial, pos)
            # the candidate set packed as a tree: same nodes, same parents, same source
            mn = rnd.choice([1, 2, 9, 24, 64])
            wt, wp, wsrc = d.draft_tree(mn)
            gt, gp, gtsrc = ts.ts_draft_tree(s, mn)
            assert (gt, gp, gtsrc) == (wt, wp[1:], wsrc), (trial, pos, mn)
            n = rnd.randrange(1, 8)
            span = script[pos:pos + n]
            used, fin = d.commit(span, v.eos, 200)
            ts.ts_commit_forced(s, span)
            info = s.state()
            assert info.n_output == len(d.y) and bool(info.finished) == fin
            assert info.fsm_kind == KIND[d.fsm.kind]
            if d.fsm.kind in (oracle.Q_P, oracle.Q_V):
                assert (info.fsm_tool, info.fsm_key) == (d.fsm.tool, d.fsm.key)
            assert info.cache_len == len(prompt) - 1 + len(d.y)
            pos += used
            if fin:
                break
        assert s.output() == d.y


def test_large_store_whole_index_search():
    schema = synth.make_schema(8192, 64, seed=9)
    inv = synth.make_datastore(schema, 3000, seed=9, total_len=(20, 120))
    d, s = _pair(schema, inv, n_cap=64)
    rnd = random.Random(9)
    hits = 0
    for trial in range(60):
        tid, toks = inv[rnd.randrange(len(inv))]
        cut = rnd.randrange(5, len(toks))
        d.y = list(toks[:cut]) if trial % 3 else [rnd.randrange(64, 8192) for _ in range(9)]
        # mirror y into the C session through forced commits on a fresh session
        s = ts.Session(None, s.schema, s.store, n_cap=64)
        ts.ts_prefill(None, s, [77])
        ts.ts_commit_forced(s, d.y)
        want, _ = oracle.suffix_match(d.y, d.store, None, 64, 63)
        got, src = ts.ts_draft(s, 63)
        wt, wp, wsrc = d.draft_tree(64)
        gt, gp, gtsrc = ts.ts_draft_tree(s, 64)
        assert (gt, gp, gtsrc) == (wt, wp[1:], wsrc)
        if want:
            hits += 1
            assert src == 2 and got == want
            assert gtsrc == 2 and gt[:len(want)] == want[:len(gt)]      # the chain draft is the first branch
        else:
            assert src != 2
    assert hits > 20


def test_session_errors():
    schema = synth.make_schema(4096, 4, seed=1)
    sc = ts.Schema(schema.vocab, schema.tools)
    s = ts.Session(None, sc, None)
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit_forced(s, [5])
    assert e.value.code == -2          # no context yet
    ts.ts_prefill(None, s, [9, 3])
    with pytest.raises(ts.TsError):
        ts.ts_prefill(None, s, [9, 3])   # twice
    assert ts.ts_draft(s, 0) == ([], 0)
    with pytest.raises(ts.TsError):
        s.set_ranks([0])                 # no datastore


@pytest.mark.parametrize("T,KB,n", [(48, 64, 148), (32, 64, 148), (192, 64, 148), (32, 192, 148), (1187, 64, 148),
                                    (6, 4, 148), (2, 4, 148), (1, 1, 148), (7, 3, 5), (5, 9, 4), (3, 64, 1)])
def test_fused_schedule_partition(T, KB, n):
    """The persistent kernel's split of a projection over CTAs: every (tile, k-block) unit exactly
    once, equal shares to within one unit among the CTAs that take part, a tile's pieces on
    consecutive CTAs, whole tiles in the middle of a range, one parked piece per slot at most."""
    L = B.lib()
    seen, sizes, per_tile = {}, [], {}
    for c in range(n):
        buf = (C.c_int32 * (6 * 4096))()
        cnt = C.c_int32()
        assert L.ts_debug_schedule(T, KB, n, c, 4096, buf, C.byref(cnt)) == 0
        segs = [tuple(buf[6 * i:6 * i + 6]) for i in range(cnt.value)]
        units, slots = 0, set()
        for i, (tile, kb0, kb1, slot, c_first, n_seg) in enumerate(segs):
            assert 0 <= tile < T and 0 <= kb0 < kb1 <= KB
            for kb in range(kb0, kb1):
                assert (tile, kb) not in seen
                seen[(tile, kb)] = c
            units += kb1 - kb0
            assert slot == (0 if i == 0 else 1)
            partial = not (kb0 == 0 and kb1 == KB)
            assert (n_seg > 1) == partial
            if partial:
                assert slot not in slots and (i == 0 or i == len(segs) - 1)
                slots.add(slot)
            per_tile.setdefault(tile, []).append((c, c_first, n_seg))
        if units:
            sizes.append(units)
    assert len(seen) == T * KB
    assert len(sizes) == min(n, T * KB) and max(sizes) - min(sizes) <= 1
    for tile, lst in per_tile.items():
        assert [c for c, _, _ in lst] == list(range(lst[0][1], lst[0][1] + lst[0][2]))
        assert all(cf == lst[0][1] and ns == lst[0][2] for _, cf, ns in lst)


def test_general_sd_drafts_bit_exact_with_oracle():
    """Context match and recycled-successor trees (host only): the same table and context on both sides."""
    schema = synth.make_schema(4096, 8, seed=4)
    rnd = random.Random(31)
    sc = ts.Schema(schema.vocab, schema.tools)
    seen = set()
    for trial in range(60):
        d = oracle.Drafter(schema, oracle.Datastore(len(schema.tools)), general_sd=True)
        s = ts.Session(None, sc, None)
        s.enable_general_sd()
        alphabet = rnd.choice([3, 50, 4000])
        prompt = [64 + rnd.randrange(alphabet) for _ in range(rnd.randint(1, 30))]     # no tool call: q_o
        d.feed_prompt(prompt)
        ts.ts_prefill(None, s, prompt)
        for step in range(12):
            # the same successor lists on both sides, for some of the tokens around
            for _ in range(rnd.randint(0, 6)):
                t = 64 + rnd.randrange(alphabet)
                ids = rnd.sample(range(64, 64 + max(alphabet, 16)), oracle.TOPK)
                d.successors[t] = ids
                s.set_successors(t, ids)
                assert s.successors(t) == ids
            mn = rnd.choice([1, 2, 7, 18, 64])
            wt, wp, wsrc = d.draft_tree(mn)
            gt, gp, gsrc = ts.ts_draft_tree(s, mn)
            assert (gt, gp, gsrc) == (wt, wp[1:], wsrc), (trial, step, mn)
            seen.add(wsrc)
            span = [64 + rnd.randrange(alphabet) for _ in range(rnd.randint(1, 4))]
            d.commit(span, schema.vocab.eos, 10 ** 6)
            ts.ts_commit_forced(s, span)
    assert {0, 3, 4} <= seen
    # off by default: the same session state drafts nothing in q_o
    s2 = ts.Session(None, sc, None)
    ts.ts_prefill(None, s2, [70, 71, 72, 73, 74, 75, 70, 71, 72, 73, 74, 75])
    assert ts.ts_draft_tree(s2, 16) == ([], [], 0)


def test_bench_tree_shapes_are_valid_trees():
    """The draft-tree shapes bench.py --tree feeds to ts_verify_tree: parents precede their children, four branches."""
    import bench
    for k in range(1, 65):
        par = bench.tree_parents(k)
        assert len(par) == k - 1
        for j, p in enumerate(par):
            assert 0 <= p <= j                         # node j + 1 hangs from an earlier node
        assert par.count(0) == min(4, sum(1 for n in (k - 1 - (k - 1) // 2, (k - 1) // 2 - (k - 1) // 4,
                                                      (k - 1) // 4 - (k - 1) // 8, (k - 1) // 8) if n > 0))
