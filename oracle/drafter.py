"""CPU oracle for the two drafters and the decode loop of Algorithm 1.

TEST INFRASTRUCTURE ONLY (see oracle/transformer.py).  Deliberately naive: linear scans, no index.

Follows, in the paper's order and notation:
  * Section 4.2 / Eq. 1: the finite-state machine F = (Q, Sigma_schema, delta, q0) with the
    tool-name state q_t, parameter-name state q_p, parameter-value state q_v and "others" state
    q_o; Eq. 2: a structural draft is prefix (+) tool_name (+) suffix; delimiters move the machine
    between q_v and q_p and close the call;
  * Section 4.3 / Eq. 4: suffix match of the generated output against historical invocations,
    suffix lengths L in {5,6,7} tried longest first, continuation y'[m : m+n);
  * Algorithm 1: retrieval has priority; the schema draft is used only when retrieval is empty.

Readings where the paper is silent (each also listed in the design notes): one candidate chain
per step; the literal scaffolding strings are fixed id tuples supplied with the schema; every
invocation carries all keys of its tool in declared order; an off-schema token drops the machine
to q_o; delta is applied token by token to every emitted token, the bonus token included; the
first hit in the order (L descending, candidate rank ascending, match position ascending) with a
non-empty continuation wins; the tool guessed in q_t is the first ranked candidate's tool that is
still compatible with the name tokens seen so far, else the compatible tool that occurs most often
in the datastore, else the lowest compatible tool id.  These choices are *parity unpinned* by the
paper: they are pinned only by the validity and brute-force tests.
"""
from typing import List, Optional, Sequence, Tuple

import numpy as np

# FSM state kinds
Q_O, Q_T, Q_P, Q_V, Q_DONE = "q_o", "q_t", "q_p", "q_v", "done"

SUFFIX_LENGTHS = (7, 6, 5)      # Appendix B.2: longest first, from 7 to 5
DEFAULT_N_CAP = 32              # Appendix B.2: first continuation length
LATER_CAPS = (16, 8, 8)         # Appendix B.2: lengths of the second to fourth continuation
MAX_TOOL_CANDIDATES = 8         # tool names verified in parallel in q_t (a reading: the paper says "all")
TOPK = 8                        # successors kept per token by the recycling drafter (a reading)
# Static tree of the recycling drafter (Appendix A.1: "a pre-defined static tree"; the shape is a reading): slots in
# breadth-first order, slot i + 1 = (parent slot, rank of the parent's successor it carries); slot 0 = pending token.
RECYCLE_TREE = ((0, 0), (0, 1), (0, 2), (0, 3), (1, 0), (1, 1), (1, 2), (2, 0), (2, 1), (3, 0),
                (4, 0), (5, 0), (5, 1), (6, 0), (8, 0), (12, 0), (16, 0))


class SchemaFsm:
    """State = (kind, stage, i, tool, key, name_prefix).

    q_t stages: 'pfx' (i scaffolding ids consumed), 'name' (name_prefix consumed), 'mid'.
    q_p stages: 'key' (i ids of key number `key` consumed), 'sep'.
    q_v stages: 'val' (free), 'nxt' / 'end' (i ids of that delimiter consumed).
    """

    def __init__(self, schema):
        self.schema = schema
        self.v = schema.vocab
        self.reset()

    def reset(self):
        self.kind, self.stage, self.i, self.tool, self.key, self.name_prefix = \
            Q_O, "", 0, -1, 0, []

    def snapshot(self):
        return (self.kind, self.stage, self.i, self.tool, self.key, tuple(self.name_prefix))

    # -- helpers -------------------------------------------------------------------------------
    def compatible_tools(self, prefix: Sequence[int]) -> List[int]:
        n = len(prefix)
        return [t for t, tool in enumerate(self.schema.tools)
                if len(tool.name) >= n and list(tool.name[:n]) == list(prefix)]

    def _to_o(self, token: int):
        self.reset()
        if token == self.v.tool_call:
            self.kind, self.stage, self.i = Q_T, "pfx", 0
            if len(self.v.pfx) == 0:
                self.stage = "name"

    def _expect(self, seq: Sequence[int], token: int) -> Optional[bool]:
        """Consume one id of a fixed string: None = mismatch, False = more to come, True = done."""
        if token != seq[self.i]:
            return None
        self.i += 1
        return self.i == len(seq)

    # -- delta ---------------------------------------------------------------------------------
    def step(self, token: int):
        v, tools = self.v, self.schema.tools
        if self.kind == Q_DONE:
            return
        if self.kind == Q_O:
            self._to_o(token)
            return
        if self.kind == Q_T:
            if self.stage == "pfx":
                r = self._expect(v.pfx, token)
                if r is None:
                    self._to_o(token)
                elif r:
                    self.stage, self.i, self.name_prefix = "name", 0, []
            elif self.stage == "name":
                exact = [t for t in self.compatible_tools(self.name_prefix)
                         if len(tools[t].name) == len(self.name_prefix)]
                if token == v.mid[0] and exact:
                    self.tool, self.stage, self.i = exact[0], "mid", 1
                    if self.i == len(v.mid):
                        self.kind, self.stage, self.i, self.key = Q_P, "key", 0, 0
                elif self.compatible_tools(self.name_prefix + [token]):
                    self.name_prefix = self.name_prefix + [token]
                else:
                    self._to_o(token)
            else:  # mid
                r = self._expect(v.mid, token)
                if r is None:
                    self._to_o(token)
                elif r:
                    self.kind, self.stage, self.i, self.key = Q_P, "key", 0, 0
            return
        if self.kind == Q_P:
            if self.stage == "key":
                r = self._expect(tools[self.tool].keys[self.key], token)
                if r is None:
                    self._to_o(token)
                elif r:
                    self.stage, self.i = "sep", 0
            else:
                r = self._expect(v.kvsep, token)
                if r is None:
                    self._to_o(token)
                elif r:
                    self.kind, self.stage, self.i = Q_V, "val", 0
            return
        # q_v
        if self.stage == "val":
            if token == v.nxt[0]:
                if self.key + 1 < len(tools[self.tool].keys):
                    self.stage, self.i = "nxt", 1
                    if self.i == len(v.nxt):
                        self.kind, self.stage, self.i, self.key = Q_P, "key", 0, self.key + 1
                else:
                    self._to_o(token)
            elif token == v.end[0]:
                self.stage, self.i = "end", 1
                if self.i == len(v.end):
                    self.kind = Q_DONE
            # any other id is part of the value
        elif self.stage == "nxt":
            r = self._expect(v.nxt, token)
            if r is None:
                self._to_o(token)
            elif r:
                self.kind, self.stage, self.i, self.key = Q_P, "key", 0, self.key + 1
        else:  # end
            r = self._expect(v.end, token)
            if r is None:
                self._to_o(token)
            elif r:
                self.kind = Q_DONE

    # -- SchemaAwareDraft ----------------------------------------------------------------------
    def draft(self, guess_tool) -> List[int]:
        """Deterministic schema filling from the current state (Eq. 2).  `guess_tool(prefix)`
        returns the tool id to assume while the name is still open."""
        v, tools = self.v, self.schema.tools
        if self.kind == Q_T:
            if self.stage == "mid":
                t = tools[self.tool]
                return list(v.mid[self.i:]) + list(t.keys[0]) + list(v.kvsep)
            prefix = [] if self.stage == "pfx" else self.name_prefix
            head = list(v.pfx[self.i:]) if self.stage == "pfx" else []
            g = guess_tool(prefix)
            if g < 0:
                return head
            t = tools[g]
            return head + list(t.name[len(prefix):]) + list(v.mid) + list(t.keys[0]) + list(v.kvsep)
        if self.kind == Q_P:
            t = tools[self.tool]
            if self.stage == "key":
                return list(t.keys[self.key][self.i:]) + list(v.kvsep)
            return list(v.kvsep[self.i:])
        if self.kind == Q_V:
            if self.stage == "nxt":
                t = tools[self.tool]
                return list(v.nxt[self.i:]) + list(t.keys[self.key + 1]) + list(v.kvsep)
            if self.stage == "end":
                return list(v.end[self.i:])
        return []


class Datastore:
    """Historical invocations y_j with the tool each one called, in insertion order."""

    def __init__(self, n_tools: int):
        self.entries: List[List[int]] = []
        self.tool_of: List[int] = []
        self.freq = [0] * n_tools

    def add(self, tokens: Sequence[int], tool_id: int):
        self.entries.append(list(tokens))
        self.tool_of.append(tool_id)
        if 0 <= tool_id < len(self.freq):
            self.freq[tool_id] += 1


def suffix_match(y: Sequence[int], store: Datastore, ranks: Optional[Sequence[int]],
                 n_cap: int, max_draft: int) -> Tuple[List[int], Tuple[int, int, int]]:
    """Eq. 4.  For L = 7, 6, 5: s = last L ids of the generated output y; candidates in rank order
    (all entries in insertion order when no rank list is installed); positions m ascending; a hit
    is y'[m-L:m] == s with m < |y'|.  Draft = y'[m : m + min(n_cap, max_draft)].
    Returns (draft, (L, candidate, m)) or ([], (0, -1, -1))."""
    order = range(len(store.entries)) if ranks is None else ranks
    n = min(n_cap, max_draft)
    if n <= 0:
        return [], (0, -1, -1)
    for L in SUFFIX_LENGTHS:
        if len(y) < L:
            continue
        s = list(y[-L:])
        for c in order:
            e = store.entries[c]
            if len(e) <= L:
                continue
            m = -1
            for mm in range(L, len(e)):
                if e[mm - L:mm] == s:
                    m = mm
                    break
            if m >= 0:
                return e[m:m + n], (L, c, m)
    return [], (0, -1, -1)


def suffix_matches(y: Sequence[int], store: Datastore, ranks: Optional[Sequence[int]],
                   caps: Sequence[int], max_draft: int) -> List[List[int]]:
    """The candidate set of retrieval drafting (Eq. 4 with Appendix B.2's continuation lengths): hits
    are taken in the order (L descending, candidate rank ascending, match position ascending); a
    position already taken at a longer L is not taken again; the i-th hit contributes
    y'[m : m + min(caps[i], max_draft)].  At most len(caps) continuations; the first one is
    suffix_match's draft."""
    order = list(range(len(store.entries))) if ranks is None else list(ranks)
    out: List[List[int]] = []
    taken = set()
    if max_draft <= 0:
        return out
    for L in SUFFIX_LENGTHS:
        if len(y) < L:
            continue
        s = list(y[-L:])
        for c in order:
            e = store.entries[c]
            if len(e) <= L:
                continue
            a = np.asarray(e)
            ok = np.ones(a.shape[0] - L, dtype=bool)
            for i in range(L):
                ok &= a[i:i + a.shape[0] - L] == s[i]
            for start in np.flatnonzero(ok):
                m = int(start) + L
                if (c, m) in taken:
                    continue
                taken.add((c, m))
                out.append(e[m:m + min(caps[len(out)], max_draft)])
                if len(out) == len(caps):
                    return out
    return out


def context_match(ctx: Sequence[int], n: int) -> List[int]:
    """Suffix match inside the context itself (prompt followed by the output), the fallback the ablation of
    Section 5.3 describes: L = 7, 6, 5 ids at the end of the context, the earliest earlier occurrence (the suffix
    matching itself excluded), continuation of at most n ids."""
    ctx = list(ctx)
    if n <= 0:
        return []
    for L in SUFFIX_LENGTHS:
        if len(ctx) <= L:
            continue
        s = ctx[-L:]
        for m in range(L, len(ctx)):
            if ctx[m - L:m] == s:
                return ctx[m:m + n]
    return []


def recycled_tree(pending: int, table: dict, max_nodes: int):
    """Static draft tree over recycled successors (Token Recycling as Section 2 describes it: the top-k
    candidates of previous steps kept per token, a tree built breadth-first).  A slot whose parent is left out
    or whose parent's token has no successor list is left out; nodes are numbered in creation order; nothing is
    added once the chunk holds max_nodes nodes.  Returns (tokens of nodes 1.., parents of all nodes)."""
    tokens: List[int] = []
    parents: List[int] = [-1]
    node_of, tok_of = {0: 0}, {0: pending}
    for i, (ps, rank) in enumerate(RECYCLE_TREE, start=1):
        if ps not in node_of or len(parents) >= max_nodes or tok_of[ps] not in table:
            continue
        t = table[tok_of[ps]][rank]
        tokens.append(int(t))
        parents.append(node_of[ps])
        node_of[i], tok_of[i] = len(parents) - 1, int(t)
    return tokens, parents


def pack_candidates(candidates: Sequence[Sequence[int]], max_nodes: int):
    """PackDraftsAsTree (Algorithm 1): merge candidate chains (each a continuation of the pending
    token) into a token trie.  Nodes are numbered in creation order, candidates inserted in the
    given order, so a parent always precedes its children; a candidate stops adding nodes once the
    chunk holds max_nodes nodes (root included).  Returns (tokens of nodes 1.., parents of all
    nodes, parents[0] = -1)."""
    tokens: List[int] = []
    parents: List[int] = [-1]
    children = [dict()]
    for cand in candidates:
        u = 0
        for t in cand:
            nxt = children[u].get(t)
            if nxt is None:
                if len(parents) >= max_nodes:
                    break
                nxt = len(parents)
                parents.append(u)
                tokens.append(int(t))
                children.append(dict())
                children[u][t] = nxt
            u = nxt
    return tokens, parents


class Drafter:
    """Per-session drafter state: FSM, generated output y, candidate rank list."""

    def __init__(self, schema, store: Datastore, n_cap: int = DEFAULT_N_CAP,
                 ranks: Optional[Sequence[int]] = None, general_sd: bool = False):
        self.schema, self.store, self.n_cap = schema, store, n_cap
        self.general_sd = general_sd        # drafts for q_v / q_o: context match, then recycled successors
        self.prompt: List[int] = []
        self.successors: dict = {}          # token -> the model's TOPK ids right after it, best first
        self.ranks = None if ranks is None else list(ranks)
        self.fsm = SchemaFsm(schema)
        self.y: List[int] = []

    def feed_prompt(self, tokens: Sequence[int]):
        self.prompt = list(tokens)
        for t in tokens:
            self.fsm.step(t)

    def update_successors(self, chunk: Sequence[int], topk_rows: Sequence[Sequence[int]]):
        """After a verification: row j was fed chunk[j]; its TOPK highest logits become that token's list."""
        for t, ids in zip(chunk, topk_rows):
            self.successors[int(t)] = [int(i) for i in ids[:TOPK]]

    def guess_tool(self, prefix: Sequence[int]) -> int:
        comp = self.fsm.compatible_tools(prefix)
        if not comp:
            return -1
        if self.ranks is not None:
            cs = set(comp)
            for c in self.ranks:
                if self.store.tool_of[c] in cs:
                    return self.store.tool_of[c]
        best = comp[0]
        for t in comp:
            if self.store.freq[t] > self.store.freq[best]:
                best = t
        return best

    def draft(self, max_draft: int) -> Tuple[List[int], int]:
        """Algorithm 1, drafting part of the loop body.  Returns (draft ids, source) with source
        0 = none, 1 = schema FSM, 2 = retrieval."""
        if max_draft <= 0:
            return [], 0
        d, _ = suffix_match(self.y, self.store, self.ranks, self.n_cap, max_draft)
        if d:
            return d, 2
        d = self.fsm.draft(self.guess_tool)[:max_draft]
        return (d, 1) if d else ([], 0)

    def draft_candidates(self, max_draft: int) -> Tuple[List[List[int]], int]:
        """The candidate set B of Algorithm 1: up to four retrieved continuations (lengths n_cap, 16,
        8, 8), else the schema drafts -- in q_t with the name still open one chain per compatible
        tool (Eq. 2: the guessed tool first, then ascending tool id, at most MAX_TOOL_CANDIDATES),
        otherwise the single deterministic chain.  The first candidate is always draft()'s chain."""
        if max_draft <= 0:
            return [], 0
        cands = suffix_matches(self.y, self.store, self.ranks, (self.n_cap,) + LATER_CAPS, max_draft)
        if cands:
            return cands, 2
        f = self.fsm
        if f.kind == Q_T and f.stage != "mid":
            prefix = [] if f.stage == "pfx" else f.name_prefix
            g = self.guess_tool(prefix)
            if g >= 0:
                order = [g] + [t for t in f.compatible_tools(prefix) if t != g]
                cands = [f.draft(lambda _p, t=t: t)[:max_draft] for t in order[:MAX_TOOL_CANDIDATES]]
                return cands, 1
        d = f.draft(self.guess_tool)[:max_draft]
        return ([d], 1) if d else ([], 0)

    def draft_tree(self, max_nodes: int) -> Tuple[List[int], List[int], int]:
        """(tokens of nodes 1.., parents of all nodes, source): the candidates packed as a trie."""
        cands, src = self.draft_candidates(max_nodes - 1)
        if not cands and self.general_sd and max_nodes > 1:
            d = context_match(self.prompt + self.y, min(self.n_cap, max_nodes - 1))
            if d:
                cands, src = [d], 3
            else:
                pending = self.y[-1] if self.y else self.prompt[-1]
                toks, par = recycled_tree(pending, self.successors, max_nodes)
                return toks, par, (4 if toks else 0)
        toks, par = pack_candidates(cands, max_nodes)
        return toks, par, (src if toks else 0)

    def commit(self, emitted: Sequence[int], eos: int, max_new_tokens: int) -> Tuple[int, bool]:
        """Append emitted ids to y one at a time, applying delta to each; stop at the first id
        that finishes the generation (call complete, EOS, or the token budget).  Returns
        (number of ids consumed, finished)."""
        n = 0
        for t in emitted:
            self.y.append(t)
            self.fsm.step(t)
            n += 1
            if self.finished(eos, max_new_tokens):
                return n, True
        return n, self.finished(eos, max_new_tokens)

    def finished(self, eos: int, max_new_tokens: int) -> bool:
        return (self.fsm.kind == Q_DONE or (len(self.y) > 0 and self.y[-1] == eos)
                or len(self.y) >= max_new_tokens)


def validate_prefix(schema, tokens: Sequence[int]) -> bool:
    """Independent check (recursive descent over the grammar, not the FSM): is `tokens` a prefix of
    the rendering of some invocation of some tool, with every key in declared order and values
    free of scaffolding ids?  Used by the tests to pin the schema drafts."""
    v = schema.vocab
    punct = set(v.pfx) | set(v.mid) | set(v.kvsep) | set(v.nxt) | set(v.end)

    def lit(pos, seq):
        """match a literal; returns new pos, or 'P' if tokens ran out while matching, or None."""
        for s in seq:
            if pos == len(tokens):
                return "P"
            if tokens[pos] != s:
                return None
            pos += 1
        return pos

    def value(pos):
        while pos < len(tokens) and tokens[pos] not in punct:
            pos += 1
        return pos

    for tool in schema.tools:
        pos = lit(0, list(v.pfx) + list(tool.name) + list(v.mid))
        if pos == "P":
            return True
        if pos is None:
            continue
        ok = True
        for ki, key in enumerate(tool.keys):
            pos = lit(pos, (list(v.nxt) if ki else []) + list(key) + list(v.kvsep))
            if pos == "P":
                return True
            if pos is None:
                ok = False
                break
            pos = value(pos)
            if pos == len(tokens):
                return True
        if not ok:
            continue
        pos = lit(pos, list(v.end))
        if pos == "P" or pos == len(tokens):
            return True
    return False
