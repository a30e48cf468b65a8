"""GPU parity tests: the CUDA verify path, called through the C ABI, against the CPU oracle on the
same seeded inputs.  Logits within max-abs 3e-2 / mean-abs 3e-3; drafts bit-exact; accepted lengths,
argmax and emitted ids exact except at positions where the oracle's top-2 logit gap is below 0.05."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from gpu_util import make_pair, synthetic_context, check_step

pytestmark = pytest.mark.gpu

# both implementations of a step: 1 = one kernel per stage, 2 = the single persistent kernel
PATHS = [pytest.param(1, id="separate"), pytest.param(2, id="fused")]


def _rand_draft(vocab, n, seed):
    g = torch.Generator().manual_seed(seed)
    return [int(x) for x in torch.randint(64, vocab, (n,), generator=g)]


def _stores(schema, inv):
    st_o, st_c = oracle.Datastore(len(schema.tools)), ts.Datastore(len(schema.tools))
    for tid, toks in inv:
        st_o.add(toks, tid)
        st_c.add(toks, tid)
    return st_o, st_c


@pytest.mark.parametrize("path", PATHS)
def test_c1_decode_loop_parity(path):
    """Config 1: tiny decoder, 256-token context through the real prefill on both sides, k = 8,
    8 tools, 64 historical invocations, 20 decode steps following the oracle's trajectory."""
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=8, max_ctx=512, path=path)
    schema = synth.make_schema(shape.vocab, 8)
    inv = synth.make_datastore(schema, 64)
    v = schema.vocab
    prompt = synth.make_context(shape.vocab, 256)
    # self-history: the model's own earlier output, once intact and once corrupted at seeded places,
    # is part of the datastore, so that retrieval drafts are accepted fully and partially
    y_ref = oracle.vanilla_greedy(om, schema, prompt, v.eos, 60)
    bad = list(y_ref)
    for p in (9, 17, 22, 40):
        bad[p] = (bad[p] + 1) % shape.vocab
    inv = inv + [(-1, bad), (-1, y_ref)]
    st_o, st_c = _stores(schema, inv)
    sc = ts.Schema(schema.vocab, schema.tools)
    d = oracle.Drafter(schema, st_o)
    d.feed_prompt(prompt)
    cache, pending = oracle.prefill(om, prompt)
    s = ts.Session(gm, sc, st_c, max_new_tokens=60)
    ts.ts_prefill(gm, s, prompt)
    assert s.state().cache_len == 255 and s.state().pending == pending
    accepted = []
    for step in range(20):
        want, src = d.draft(7)
        got, gsrc = ts.ts_draft(s, 7)
        assert (got, gsrc) == (want, src)
        n0 = cache.length
        ref = om.verify(pending, want, cache, want_logits=True)
        res = ts.ts_verify(gm, [s], [got])[0]
        assert res.k == len(want) + 1
        check_step(res, gm.read_logits(0, res.k), ref, f"step {step}")
        used, fin = d.commit(ref["emitted"], v.eos, 60)
        cache.truncate(n0 + used)
        ts.ts_commit_forced(s, ref["emitted"])          # re-synchronise on the oracle's trajectory
        pending = ref["emitted"][used - 1]
        info = s.state()
        assert (info.cache_len, info.pending, bool(info.finished)) == (cache.length, pending, fin)
        accepted.append(ref["accept_len"])
        if fin:
            break
    assert s.output() == d.y == y_ref[:len(d.y)]
    assert max(accepted) == 7 and 0 < min(a for a in accepted if a) < 7   # full and partial acceptance


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,ctx,k", [("1b-2l", 128, 4), ("1b-2l", 128, 8), ("1b-2l", 131, 16), ("8b-2l", 100, 32)])
def test_real_prefill_shapes(name, ctx, k, path):
    """Configs 2/3 at reduced depth: real prefill on both sides (K/V are rounded to bf16 on the
    GPU only), then one verify step with a partly correct draft."""
    shape = synth.SHAPES[name]
    om, gm = make_pair(shape, k_max=max(k, 16), max_ctx=512, path=path)
    prompt = synth.make_context(shape.vocab, ctx)
    cache, pending = oracle.prefill(om, prompt)
    s = ts.Session(gm, None, None)
    ts.ts_prefill(gm, s, prompt)
    truth, c2, p2 = [], cache.clone(), pending
    for _ in range(3):
        p2 = om.greedy_next(p2, c2)
        truth.append(p2)
    draft = (truth + _rand_draft(shape.vocab, k, 3))[:k - 1]
    ref = om.verify(pending, draft, cache, want_logits=True)
    res = ts.ts_verify(gm, [s], [draft])[0]
    check_step(res, gm.read_logits(0, k), ref, f"{name} k={k}")
    gm.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,ctx,k", [("8b-2l", 2048, 32), ("8b-2l", 1000, 1), ("8b-2l", 64, 17),
                                        ("1b-2l", 4096, 16), ("1b-2l", 15, 2), ("tiny", 0, 8), ("8b-2l", 700, 64)])
def test_synthetic_kv_single(name, ctx, k, path):
    """Long contexts as seeded synthetic K/V imported on both sides; ragged lengths around page and
    block boundaries; k = 1 (empty draft) and an empty cache included."""
    shape = synth.SHAPES[name]
    om, gm = make_pair(shape, k_max=max(k, 8), max_ctx=ctx + 64, path=path)
    cache, s, pending = synthetic_context(shape, om, gm, ctx)
    draft = _rand_draft(shape.vocab, k - 1, 5)
    ref = om.verify(pending, draft, cache, want_logits=True)
    res = ts.ts_verify(gm, [s], [draft])[0]
    check_step(res, gm.read_logits(0, k), ref, f"{name} ctx={ctx} k={k}")
    # the step is idempotent until committed: a replay reproduces the logits bit for bit
    a = gm.read_logits(0, k).copy()
    ts.ts_verify_replay(gm)
    torch.cuda.synchronize()
    assert np.array_equal(a, gm.read_logits(0, k))
    # commit, then a second step sees the accepted rows in the cache
    ts.ts_commit(s, res)
    cache.truncate(ctx + res.n_emitted)
    if res.accept_len == ref["accept_len"] and list(res.emitted[:res.n_emitted]) == ref["emitted"]:
        d2 = _rand_draft(shape.vocab, min(3, k), 6)
        ref2 = om.verify(ref["emitted"][-1], d2, cache, want_logits=True)
        res2 = ts.ts_verify(gm, [s], [d2])[0]
        check_step(res2, gm.read_logits(0, len(d2) + 1), ref2, "second step")
    gm.close()


def test_ragged_batch():
    """Config-4-like: several sessions with ragged contexts and per-sequence k in one batched step
    (more than 128 rows, so the GEMMs run several row chunks)."""
    shape = synth.SHAPES["8b-2l"]
    lens = [70, 333, 1024, 129, 640, 2047]
    ks = [32, 4, 29, 17, 32, 30]
    om, gm = make_pair(shape, max_batch=6, k_max=32, max_rows=sum(ks), max_ctx=2048 + 64)
    sess, caches, drafts, refs = [], [], [], []
    for i, (n, k) in enumerate(zip(lens, ks)):
        cache, s, pending = synthetic_context(shape, om, gm, n, stream=i, pending=100 + i)
        draft = _rand_draft(shape.vocab, k - 1, 10 + i)
        sess.append(s); caches.append(cache); drafts.append(draft)
        refs.append(om.verify(pending, draft, cache, want_logits=True))
    out = ts.ts_verify(gm, sess, drafts)
    row = 0
    for i, (res, ref) in enumerate(zip(out, refs)):
        assert res.first_row == row and res.k == ks[i]
        check_step(res, gm.read_logits(row, res.k), ref, f"seq {i}")
        row += res.k
    gm.close()


@pytest.mark.parametrize("name", ["8b-2l", "1b-2l"])
@pytest.mark.parametrize("ks", [[32, 32, 1], [40, 33, 30], [64, 64], [64, 64, 1], [64, 64, 64, 64], [33, 64, 64, 64, 64, 11]],
                         ids=lambda ks: f"{sum(ks)}rows")
def test_row_counts_around_the_projection_kernels_switch(name, ks):
    """Steps of 65, 103, 128, 129, 256 and 300 rows: the first size past the weight-streaming projection kernel, one
    partly filled 128-row chunk, exactly one chunk, one row into a second chunk, two full chunks (the case in which the
    many-rows kernel mixes tile widths and cuts K by its cost model), and three chunks with a ragged last one."""
    shape = synth.SHAPES[name]
    lens = [70, 333, 1024, 129, 640, 17][:len(ks)]
    om, gm = make_pair(shape, max_batch=len(ks), k_max=64, max_rows=sum(ks), max_ctx=1024 + 128)
    sess, drafts, refs = [], [], []
    for i, (n, k) in enumerate(zip(lens, ks)):
        cache, s, pending = synthetic_context(shape, om, gm, n, stream=i, pending=300 + i)
        draft = _rand_draft(shape.vocab, k - 1, 70 + i)
        sess.append(s); drafts.append(draft)
        refs.append(om.verify(pending, draft, cache, want_logits=True))
    out = ts.ts_verify(gm, sess, drafts)
    row = 0
    for i, (res, ref) in enumerate(zip(out, refs)):
        assert res.first_row == row and res.k == ks[i]
        check_step(res, gm.read_logits(row, res.k), ref, f"{name}, {sum(ks)} rows, seq {i}")
        row += res.k
    gm.close()


def test_sixteen_sessions_512_rows():
    """The largest step of the batched configuration: 16 sessions x k = 32 = 512 rows (four 128-row chunks in every
    projection, 16 attention row tiles), ragged contexts from a few tokens to two thousand."""
    shape = synth.SHAPES["8b-2l"]
    g = np.random.Generator(np.random.Philox(key=[260413519, 0x512]))
    lens = [int(x) for x in g.integers(3, 2048, size=16)]
    lens[3], lens[11] = 2047, 16
    om, gm = make_pair(shape, max_batch=16, k_max=32, max_rows=512, max_ctx=2048 + 64)
    sess, drafts, refs = [], [], []
    for i, n in enumerate(lens):
        cache, s, pending = synthetic_context(shape, om, gm, n, stream=i, pending=200 + i)
        draft = _rand_draft(shape.vocab, 31, 40 + i)
        sess.append(s); drafts.append(draft)
        refs.append(om.verify(pending, draft, cache, want_logits=True))
    out = ts.ts_verify(gm, sess, drafts)
    for i, (res, ref) in enumerate(zip(out, refs)):
        assert res.first_row == 32 * i and res.k == 32
        check_step(res, gm.read_logits(32 * i, 32), ref, f"seq {i} (ctx {lens[i]})")
    gm.close()


def test_retrieval_heavy_batch():
    """Config-5-like: batch 4, long retrieved drafts (k = 64) from a large store searched through
    the n-gram index; drafts bit-exact with the oracle's linear scan."""
    shape = synth.SHAPES["8b-2l"]
    schema = synth.make_schema(shape.vocab, 64, seed=5)
    inv = synth.make_datastore(schema, 2000, seed=5, total_len=(20, 200))
    st_o, st_c = _stores(schema, inv)
    sc = ts.Schema(schema.vocab, schema.tools)
    om, gm = make_pair(shape, max_batch=4, k_max=64, max_ctx=1024)
    sess, drafts, refs = [], [], []
    for i in range(4):
        cache, s, pending = synthetic_context(shape, om, gm, 500 + 37 * i, stream=i, schema=sc, store=st_c, n_cap=64)
        d = oracle.Drafter(schema, st_o, n_cap=64)
        d.feed_prompt([pending])
        tid, toks = max(inv[10 * i:10 * i + 10], key=lambda e: len(e[1]))
        d.commit(toks[:12], schema.vocab.eos, 10 ** 6)
        ts.ts_verify(gm, [s], [toks[:11]])    # (a commit is checked against the chunk of the last verification)
        ts.ts_commit_forced(s, toks[:12])     # 12 generated ids
        want, src = d.draft(63)
        got, gsrc = ts.ts_draft(s, 63)
        assert (got, gsrc) == (want, src) and src == 2
        # the oracle cache must hold the same 12 extra positions: extend it with the same K/V the GPU will see
        sess.append(s); drafts.append(got)
        refs.append((cache, toks[11], want, 500 + 37 * i))
    # the oracle side never saw those 12 rows; reset both sides to the imported context
    for s, (cache, p, want, n) in zip(sess, refs):
        s.set_cache(n, p)
    out = ts.ts_verify(gm, sess, drafts)
    row = 0
    for i, res in enumerate(out):
        cache, p, want, n = refs[i]
        ref = om.verify(p, want, cache, want_logits=True)
        check_step(res, gm.read_logits(row, res.k), ref, f"seq {i}")
        row += res.k
    gm.close()


def test_argument_and_capacity_errors():
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=4, max_ctx=64, max_pages=3)
    s = ts.Session(gm, None, None)
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify(gm, [s], [[70]])
    assert e.value.code == -2                      # no context yet
    ts.ts_prefill(gm, s, [70, 71, 72])
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify(gm, [s], [[70, 71, 72, 73]])  # 5 rows > k_max
    assert e.value.code == -4
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify(gm, [s], [[shape.vocab]])
    assert e.value.code == -5
    s2 = ts.Session(gm, None, None)
    with pytest.raises(ts.TsError) as e:
        ts.ts_prefill(gm, s2, list(range(70, 70 + 40)))   # needs 3 pages, only 2 are left
    assert e.value.code == -3
    res = ts.ts_verify(gm, [s], [[70]])[0]                 # the context is still usable
    assert res.k == 2
    gm.close()


def test_commit_is_checked_against_the_verified_chunk():
    """A commit moves the cache length over rows the last verification wrote: it is refused without one, twice for
    the same one, for more ids than rows, and for ids other than the ones those rows were computed from."""
    shape = synth.SHAPES["tiny"]
    om, gm = make_pair(shape, k_max=8, max_ctx=128)
    s = ts.Session(gm, None, None)
    ts.ts_prefill(gm, s, [70, 71, 72, 73])
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit_forced(s, [80])                       # nothing verified yet
    assert e.value.code == -2
    draft = [90, 91, 92]
    res = ts.ts_verify(gm, [s], [draft])[0]
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit_forced(s, [90, 91, 92, 93, 94])       # 5 ids, 4 rows
    assert e.value.code == -1
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit_forced(s, [90, 99, 5])                # row 2 was fed 91, not 99
    assert e.value.code == -1
    assert s.state().cache_len == 3                        # the refused calls changed nothing
    ts.ts_commit_forced(s, [90, 91, 5])                    # two verified drafts kept, a free last id
    assert (s.state().cache_len, s.state().pending) == (6, 5)
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit(s, res)                               # the same verification a second time
    assert e.value.code == -2
    res = ts.ts_verify(gm, [s], [[]])[0]
    ts.ts_commit(s, res)
    assert s.state().cache_len == 7
    s.set_cache(3, 73)
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit(s, res)                               # the context was replaced since
    assert e.value.code == -2
    gm.close()


@pytest.mark.parametrize("path", PATHS)
def test_device_timeout_is_reported_and_survived(path):
    """The host's handling of an expired device-side wait, without making the GPU wait: the status word is written on
    the stream after the step's last kernel (no kernel sees it).  The step fails with TS_ERR_DEVICE_TIMEOUT, the
    session is untouched, and the next step is parity-green again."""
    shape = synth.SHAPES["1b-2l"]
    om, gm = make_pair(shape, k_max=16, max_ctx=512, path=path)
    cache, s, pending = synthetic_context(shape, om, gm, 200)
    draft = _rand_draft(shape.vocab, 9, 31)
    ref = om.verify(pending, draft, cache.clone(), want_logits=True)
    check_step(ts.ts_verify(gm, [s], [draft])[0], gm.read_logits(0, 10), ref, "before")
    gm.inject_device_error(3)
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify(gm, [s], [draft])
    assert e.value.code == -6 and "code 3" in str(e.value)
    assert (s.state().cache_len, s.state().pending) == (200, pending)
    with pytest.raises(ts.TsError) as e:
        ts.ts_commit_forced(s, ref["emitted"])            # a failed step leaves nothing to commit
    assert e.value.code == -2
    res = ts.ts_verify(gm, [s], [draft])[0]               # the word was cleared: the same step again, clean
    check_step(res, gm.read_logits(0, 10), ref, "after the reported timeout")
    ts.ts_commit(s, res)
    gm.close()


def test_device_index_check_is_reported_and_survived():
    """The host's handling of a failed index check of the debug build, exercised the same way (a status word written
    after the step's last kernel; the release build's kernels contain no checks): TS_ERR_DEVICE_BOUNDS with the check's
    number, session untouched, next step clean."""
    shape = synth.SHAPES["1b-2l"]
    om, gm = make_pair(shape, k_max=16, max_ctx=512)
    cache, s, pending = synthetic_context(shape, om, gm, 200)
    draft = _rand_draft(shape.vocab, 9, 31)
    ref = om.verify(pending, draft, cache.clone(), want_logits=True)
    gm.inject_device_error(64 + 4)
    with pytest.raises(ts.TsError) as e:
        ts.ts_verify(gm, [s], [draft])
    assert e.value.code == -9 and "check 4" in str(e.value)
    assert (s.state().cache_len, s.state().pending) == (200, pending)
    check_step(ts.ts_verify(gm, [s], [draft])[0], gm.read_logits(0, 10), ref, "after the reported index check")
    gm.close()


def test_small_batch_fused():
    """Several short sequences in one step of the persistent kernel (ragged k, ragged contexts)."""
    shape = synth.SHAPES["1b-2l"]
    lens, ks = [40, 333, 17, 129], [9, 4, 16, 11]
    om, gm = make_pair(shape, max_batch=4, k_max=16, max_rows=sum(ks), max_ctx=512, path=2)
    sess, drafts, refs = [], [], []
    for i, (n, k) in enumerate(zip(lens, ks)):
        cache, s, pending = synthetic_context(shape, om, gm, n, stream=i, pending=100 + i)
        draft = _rand_draft(shape.vocab, k - 1, 20 + i)
        sess.append(s); drafts.append(draft)
        refs.append(om.verify(pending, draft, cache, want_logits=True))
    out = ts.ts_verify(gm, sess, drafts)
    row = 0
    for i, (res, ref) in enumerate(zip(out, refs)):
        assert res.first_row == row and res.k == ks[i]
        check_step(res, gm.read_logits(row, res.k), ref, f"seq {i}")
        row += res.k
    gm.close()
