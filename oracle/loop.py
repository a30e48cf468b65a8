"""CPU oracle for the decode loop of Algorithm 1 and for vanilla greedy decoding.

TEST INFRASTRUCTURE ONLY (see oracle/transformer.py).

Algorithm 1's loop body, one candidate chain per step: draft (retrieval, else schema) -> pack the
chunk [pending, drafts] -> one verification forward -> longest accepted prefix + bonus token ->
append -> FSM update.  The vanilla loop takes one argmax per forward and uses the same stopping
rule, so the two outputs can be compared token for token (the method preserves the target
model's output: Section 5.2, Table 5).
"""
from typing import List, Optional, Sequence

from .transformer import OracleModel
from .drafter import Drafter, Datastore


def prefill(model: OracleModel, prompt: Sequence[int], chunk: int = 64):
    """Cache holding prompt[:-1]; the last prompt id is left pending."""
    cache = model.new_cache()
    body = list(prompt[:-1])
    for i in range(0, len(body), chunk):
        model.forward_chunk(body[i:i + chunk], cache)
    return cache, prompt[-1]


def vanilla_greedy(model: OracleModel, schema, prompt: Sequence[int], eos: int,
                   max_new_tokens: int, cache=None, pending=None) -> List[int]:
    if cache is None:
        cache, pending = prefill(model, prompt)
    d = Drafter(schema, Datastore(len(schema.tools)))
    d.feed_prompt(prompt)
    while not d.finished(eos, max_new_tokens):
        t = model.greedy_next(pending, cache)
        d.commit([t], eos, max_new_tokens)
        pending = t
    return d.y


def speculative_decode(model: OracleModel, schema, store: Datastore, prompt: Sequence[int],
                       eos: int, max_new_tokens: int, k_max: int, n_cap: int = 32,
                       ranks: Optional[Sequence[int]] = None, cache=None, pending=None,
                       max_steps: Optional[int] = None, trace: Optional[list] = None) -> List[int]:
    """Returns y.  `trace` (if given) receives one dict per step: pending, draft, source,
    accept_len, emitted, consumed."""
    if cache is None:
        cache, pending = prefill(model, prompt)
    d = Drafter(schema, store, n_cap=n_cap, ranks=ranks)
    d.feed_prompt(prompt)
    steps = 0
    while not d.finished(eos, max_new_tokens) and (max_steps is None or steps < max_steps):
        draft, source = d.draft(k_max - 1)
        n0 = cache.length
        res = model.verify(pending, draft, cache)
        consumed, _fin = d.commit(res["emitted"], eos, max_new_tokens)
        cache.truncate(n0 + consumed)
        if trace is not None:
            trace.append(dict(pending=pending, draft=list(draft), source=source,
                              accept_len=res["accept_len"], emitted=list(res["emitted"]),
                              consumed=consumed, argmax=list(res["argmax"])))
        pending = res["emitted"][consumed - 1]
        steps += 1
    return d.y


def speculative_decode_tree(model: OracleModel, schema, store: Datastore, prompt: Sequence[int],
                            eos: int, max_new_tokens: int, max_nodes: int, n_cap: int = 32,
                            ranks: Optional[Sequence[int]] = None, cache=None, pending=None,
                            max_steps: Optional[int] = None, trace: Optional[list] = None,
                            general_sd: bool = False) -> List[int]:
    """Algorithm 1 with its candidate set: draft candidates -> PackDraftsAsTree -> one verification
    forward under the tree mask -> longest accepted path + bonus token -> append -> FSM update.
    With general_sd the open-ended states draft too (context match, recycled successors), and every
    verification refreshes the successor lists from the per-row top-k of its logits."""
    from .tree import verify_tree
    from .transformer import topk_lowest
    from .drafter import TOPK
    if cache is None:
        cache, pending = prefill(model, prompt)
    d = Drafter(schema, store, n_cap=n_cap, ranks=ranks, general_sd=general_sd)
    d.feed_prompt(prompt)
    steps = 0
    while not d.finished(eos, max_new_tokens) and (max_steps is None or steps < max_steps):
        toks, par, source = d.draft_tree(max_nodes)
        n0 = cache.length
        res = verify_tree(model, pending, toks, par, cache, want_logits=general_sd)
        if general_sd:
            d.update_successors([pending] + list(toks), [topk_lowest(row, TOPK) for row in res["logits"]])
        consumed, _fin = d.commit(res["emitted"], eos, max_new_tokens)
        cache.truncate(n0 + consumed)
        if trace is not None:
            trace.append(dict(pending=pending, tokens=list(toks), parents=list(par), source=source,
                              accept_len=res["accept_len"], emitted=list(res["emitted"]),
                              consumed=consumed, path=list(res["path"])))
        pending = res["emitted"][consumed - 1]
        steps += 1
    return d.y
