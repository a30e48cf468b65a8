"""Seeded synthetic tool schemas, historical invocations and contexts.

The shape of the data follows the paper's description of tool-call traces: a JSON object with a
"name" and a "parameters" map (Section 3.2, Figure 4 caption), fixed scaffolding tokens, tool and
parameter names from a finite schema, free parameter values, and heavy reuse of a few tools
(Table 2).  Only token-id sequences are produced here; no drafting or matching logic.
"""
from dataclasses import dataclass, field
from typing import List, Sequence

import numpy as np

from .shapes import MASTER_SEED


@dataclass(frozen=True)
class Vocab:
    """Id layout.  Punctuation strings are fixed id tuples disjoint from every name/value id."""
    size: int
    bos: int = 1
    eos: int = 2
    tool_call: int = 3          # <tool_call>
    tool_call_end: int = 4      # </tool_call>
    pfx: tuple = (8, 9, 10)             # {"name": "
    mid: tuple = (11, 12, 13, 14)       # ", "parameters": {"
    kvsep: tuple = (15, 16)             # ": "
    nxt: tuple = (17, 18)               # ", "
    end: tuple = (19, 20)               # "}}
    first_free: int = 64                # ids below are specials / punctuation

    @property
    def name_lo(self):
        return self.first_free

    @property
    def name_hi(self):
        return self.size // 2           # names and keys in [64, V/2)

    @property
    def value_lo(self):
        return self.size // 2           # values in [V/2, V)


@dataclass
class Tool:
    name: List[int]
    keys: List[List[int]]


@dataclass
class Schema:
    vocab: Vocab
    tools: List[Tool] = field(default_factory=list)


def _rng(seed, *stream):
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ 0x7001, hash_stream(stream)]))


def hash_stream(stream) -> int:
    h = 1469598103934665603
    for s in stream:
        for ch in str(s).encode():
            h = ((h ^ ch) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
        h = ((h ^ 0xFF) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    return h


def make_schema(vocab_size: int, n_tools: int, seed: int = MASTER_SEED, name_len=(2, 4),
                n_keys=(1, 4), key_len=(1, 3), shared_name_prefix: float = 0.25) -> Schema:
    """n_tools tools with distinct names.  With probability `shared_name_prefix` a tool's name
    starts with the first token of an earlier tool's name, so that the tool-name state has real
    ambiguity to resolve."""
    v = Vocab(vocab_size)
    g = _rng(seed, "schema", vocab_size, n_tools)
    tools, seen = [], set()
    while len(tools) < n_tools:
        ln = int(g.integers(name_len[0], name_len[1] + 1))
        name = [int(x) for x in g.integers(v.name_lo, v.name_hi, size=ln)]
        if tools and g.random() < shared_name_prefix:
            name[0] = tools[int(g.integers(0, len(tools)))].name[0]
        if tuple(name) in seen:
            continue
        seen.add(tuple(name))
        nk = int(g.integers(n_keys[0], n_keys[1] + 1))
        keys = []
        for _ in range(nk):
            kl = int(g.integers(key_len[0], key_len[1] + 1))
            keys.append([int(x) for x in g.integers(v.name_lo, v.name_hi, size=kl)])
        tools.append(Tool(name, keys))
    return Schema(v, tools)


def render_invocation(schema: Schema, tool_id: int, values: Sequence[Sequence[int]]) -> List[int]:
    """Token ids of `{"name": "<tool>", "parameters": {"<k1>": "<v1>", ...}}` in the id layout."""
    v, t = schema.vocab, schema.tools[tool_id]
    assert len(values) == len(t.keys)
    out = list(v.pfx) + list(t.name) + list(v.mid)
    for i, (key, val) in enumerate(zip(t.keys, values)):
        if i:
            out += list(v.nxt)
        out += list(key) + list(v.kvsep) + list(val)
    out += list(v.end)
    return out


def zipf_tool_ids(n_tools: int, n: int, g, a: float = 1.1):
    p = 1.0 / np.arange(1, n_tools + 1) ** a
    p /= p.sum()
    return g.choice(n_tools, size=n, p=p)


def make_datastore(schema: Schema, n_inv: int, seed: int = MASTER_SEED, value_len=(1, 6),
                   total_len=None, pool_size: int = 8, p_pool: float = 0.7):
    """Historical invocations: list of (tool_id, token list).  Tools are drawn Zipf(1.1); each
    value comes with probability p_pool from a small per-(tool,key) pool (recurring arguments),
    else fresh.  If total_len=(lo,hi) is given, value lengths are stretched/resampled until the
    whole invocation has a length in that range."""
    v = schema.vocab
    g = _rng(seed, "datastore", v.size, len(schema.tools), n_inv)
    pools = {}
    out = []
    tool_ids = zipf_tool_ids(len(schema.tools), n_inv, g)
    for tid in tool_ids:
        tid = int(tid)
        tool = schema.tools[tid]
        for _attempt in range(64):
            vals = []
            for ki in range(len(tool.keys)):
                if total_len is None:
                    ln = int(g.integers(value_len[0], value_len[1] + 1))
                else:
                    fixed = len(v.pfx) + len(tool.name) + len(v.mid) + len(v.end) \
                        + sum(len(k) + len(v.kvsep) for k in tool.keys) \
                        + len(v.nxt) * (len(tool.keys) - 1)
                    budget_lo = max(1, (total_len[0] - fixed + len(tool.keys) - 1) // len(tool.keys))
                    budget_hi = max(budget_lo, (total_len[1] - fixed) // len(tool.keys))
                    ln = int(g.integers(budget_lo, budget_hi + 1))
                pool = pools.setdefault((tid, ki), [])
                if pool and g.random() < p_pool:
                    val = pool[int(g.integers(0, len(pool)))]
                else:
                    val = [int(x) for x in g.integers(v.value_lo, v.size, size=ln)]
                    if len(pool) < pool_size:
                        pool.append(val)
                vals.append(val)
            toks = render_invocation(schema, tid, vals)
            if total_len is None or total_len[0] <= len(toks) <= total_len[1]:
                break
        out.append((tid, toks))
    return out


def make_context(vocab_size: int, length: int, seed: int = MASTER_SEED, stream=0) -> List[int]:
    """`length` prompt tokens: uniform ids in [64, V), the last one being <tool_call>."""
    v = Vocab(vocab_size)
    g = _rng(seed, "context", vocab_size, length, stream)
    toks = [int(x) for x in g.integers(v.first_free, v.size, size=length)]
    toks[-1] = v.tool_call
    return toks


def planted_accept_lengths(n: int, seed: int = MASTER_SEED, stream=0, cap: int = 33):
    """Accepted-length profile with the paper's shape (mean about 5 emitted tokens per step,
    roughly 22% of steps above 8 and 4% in 17..33; Section 5.3 and Figure 8's description).
    Returns the number of *draft* tokens to leave uncorrupted at each of n steps."""
    g = _rng(seed, "accept", n, stream)
    u = g.random(n)
    out = np.empty(n, dtype=np.int64)
    for i, x in enumerate(u):
        if x < 0.04:
            out[i] = int(g.integers(16, cap))        # 17..33 emitted
        elif x < 0.22:
            out[i] = int(g.integers(8, 16))          # 9..16 emitted
        else:
            out[i] = int(g.integers(0, 8))           # 1..8 emitted
    return [int(x) for x in out]
