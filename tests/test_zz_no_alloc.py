"""ts_attention_static against the oracle's attention and against ts_verify's own attention stage.

Some users of the library cannot allocate device memory (a plugin inside a server whose memory pool
belongs to the host application, code running under a fixed memory budget), so they cannot provide
the workspace a model needs.  ts_attention_static keeps its scratch in an array inside the library
image instead.  This test feeds it what ts_verify's attention stage saw in the last layer of a step
(the rotated queries and the layer's cache, re-paged under a shuffled block table in buffers the test
owns) and requires (a) the oracle's attention of the same queries, keys and values, (b) the output of
ts_verify's attention stage, a different kernel, on two different problems in a row so that whatever
the first call leaves in the shared scratch must not leak into the second, and (c) that the device's
free memory and torch's allocation count are the same before and after the call.

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import pytest
import torch

import oracle
import synth
import paper_2604_13519_b200 as ts
from gpu_util import make_pair, synthetic_context

pytestmark = pytest.mark.gpu

TOL = 1e-3         # against ts_verify's attention stage, on outputs of magnitude ~0.1
ORACLE_TOL = 2e-3  # against the float64 oracle: softmax weights carry 11 bits (fp16), values are N(0,1)


def _own_pages(shape, sess, layer, n_tokens, seed):
    """The session's cache rows of one layer, re-paged in buffers owned by the test."""
    k, v = sess.export_kv(layer, n_tokens)                     # float32 [n][Hkv][hd], exact fp16 values
    n_pages = (n_tokens + 15) // 16
    g = torch.Generator().manual_seed(seed)
    table = torch.randperm(n_pages + 3, generator=g)[:n_pages].to(torch.int32)     # shuffled, with unused ids
    pad = n_pages * 16 - n_tokens
    kp = torch.zeros(n_pages + 3, shape.n_kv_heads, 16, shape.head_dim, dtype=torch.float16)
    vp = torch.zeros_like(kp)
    for src, dst in ((k, kp), (v, vp)):
        x = torch.cat([src, torch.zeros(pad, *src.shape[1:])]).view(n_pages, 16, shape.n_kv_heads, shape.head_dim)
        dst[table.long()] = x.permute(0, 2, 1, 3).to(torch.float16)
    return kp.cuda(), vp.cuda(), table.view(1, -1).cuda()


def _compare(shape, gm, sess, ctx, k, seed, first_call=False):
    R = (gm.cfg.max_rows + 127) // 128 * 128
    Nq = shape.n_q_heads * shape.head_dim
    q = gm.read_buffer(2)[:k].cuda().contiguous()                       # fp16 [k][Nq], last layer
    want = gm.read_buffer(3).float().sum(0)[:k]                         # hi + lo planes
    kp, vp, table = _own_pages(shape, sess, shape.n_layers - 1, ctx + k, seed)
    out = torch.zeros(2, R, Nq, dtype=torch.bfloat16, device="cuda")
    d_cu = torch.tensor([0, k], dtype=torch.int32, device="cuda")
    d_len = torch.tensor([ctx], dtype=torch.int32, device="cuda")
    # every input exists now: the call itself must not take device memory, from the driver or from torch's pool
    torch.cuda.synchronize()
    free0, alloc0, resv0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    ts.ts_attention_static(q, kp, vp, table, [0, k], [ctx], shape.n_q_heads, shape.n_kv_heads, shape.head_dim, out,
                           cu_rows_dev=d_cu, seq_len_dev=d_len)
    torch.cuda.synchronize()
    # (the driver loads a kernel's code at its first launch in a process, which can move the free-memory figure once)
    assert first_call or torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == resv0
    got = out.float().sum(0)[:k].cpu()
    err = (got - want).abs().max().item()
    assert want.abs().max().item() > 1e-3                               # the reference is not trivially zero
    assert err <= TOL, f"ctx={ctx} k={k}: max abs difference from ts_verify's attention {err:.3e}"
    # the oracle's attention over the same fp16 queries and the cache rows as exported (chunk rows included)
    kk, vv = sess.export_kv(shape.n_layers - 1, ctx + k)
    ref = oracle.attention(q.cpu().double().view(k, shape.n_q_heads, shape.head_dim), kk.double(), vv.double(),
                           torch.arange(k) + ctx, torch.arange(ctx + k)).reshape(k, Nq)
    err_o = (got.double() - ref).abs().max().item()
    assert err_o <= ORACLE_TOL, f"ctx={ctx} k={k}: max abs difference from the oracle {err_o:.3e}"


def test_static_attention_matches_verify_twice():
    shape = synth.SHAPES["8b-2l"]
    om, gm = make_pair(shape, k_max=32, max_ctx=1024)
    # first problem: 700 cached tokens, 32 rows (two 64-row tiles of packed rows, several KV splits)
    cache, sess, pending = synthetic_context(shape, om, gm, 700)
    draft = [100 + 3 * j for j in range(31)]
    ts.ts_verify(gm, [sess], [draft])
    _compare(shape, gm, sess, 700, 32, seed=1, first_call=True)
    # second problem, right after: shorter context, ragged chunk, fewer splits
    sess2_cache, sess2, _ = synthetic_context(shape, om, gm, 85, stream=1)
    draft2 = [200 + 5 * j for j in range(6)]
    ts.ts_verify(gm, [sess2], [draft2])
    _compare(shape, gm, sess2, 85, 7, seed=2)
    gm.close()


def test_static_attention_rejects_oversize():
    q = torch.zeros(1, dtype=torch.float16, device="cuda")
    table = torch.zeros(1, 4096, dtype=torch.int32, device="cuda")
    out = torch.zeros(2, 128, 1 << 17, dtype=torch.bfloat16, device="cuda")
    # 64 rows x 1024 heads x 128 x 4 bytes = 32 MiB per split: more than the 16 MiB array
    with pytest.raises(ts.TsError) as e:
        ts.ts_attention_static(q, q, q, table, [0, 64], [1000], 1024, 8, 128, out)
    assert e.value.code == -4 and "static scratch" in str(e.value)
    with pytest.raises(ts.TsError) as e:
        ts.ts_attention_static(q, q, q, table, [0, 65], [1000], 32, 8, 128, out)     # more than TS_K_MAX rows
    assert e.value.code == -4
