"""CPU oracle for tree verification: several candidate drafts verified in one forward pass.

TEST INFRASTRUCTURE ONLY (see oracle/transformer.py).

Paper: Appendix A.1 "Parallel Verification" (the candidates are compacted into one flattened
sequence and verified in a single forward pass under a tree-structured attention mask) and
Algorithm 1, steps PackDraftsAsTree / Verification / SelectLongestAcceptedPrefix.

Conventions.  A chunk of k nodes: node 0 is the pending token (the root), node j > 0 is a draft
token with parent[j] < j; parent[0] = -1.  A node attends to the cached prefix and to its ancestors
and itself; its rotary position is (cache length + depth).  Greedy acceptance walks from the root:
at node u the model's token is t_u = argmax(logits_u); the walk moves to the child of u whose
token equals t_u (the lowest-numbered one if a malformed tree has several) and stops when there
is none.  The accepted path's tokens plus the model's token at the last node are emitted; the cache
keeps the K/V rows of the path's nodes, in path order.  A chain (parent[j] = j - 1) is the ordinary
speculative step.
"""
from typing import List, Sequence

import torch

from .transformer import OracleModel, KVCache, argmax_lowest, F64
from .drafter import pack_candidates  # noqa: F401  (PackDraftsAsTree lives with the drafters)


def check_parents(parents: Sequence[int]):
    assert len(parents) >= 1 and parents[0] == -1
    for j in range(1, len(parents)):
        assert 0 <= parents[j] < j, "parents must point to an earlier node"


def node_depths(parents: Sequence[int]) -> List[int]:
    d = [0] * len(parents)
    for j in range(1, len(parents)):
        d[j] = d[parents[j]] + 1
    return d


def ancestor_mask(parents: Sequence[int]) -> torch.Tensor:
    """[k, k] bool: entry (j, i) is true iff node i is node j or one of its ancestors."""
    k = len(parents)
    m = torch.zeros(k, k, dtype=torch.bool)
    for j in range(k):
        u = j
        while u >= 0:
            m[j, u] = True
            u = parents[u]
    return m


def forward_tree(model: OracleModel, z: Sequence[int], parents: Sequence[int], cache: KVCache):
    """Logits [k, V] of all nodes and the nodes' K/V per layer; the cache is not modified."""
    check_parents(parents)
    s = model.s
    n0, k = cache.length, len(z)
    pos = torch.tensor(node_depths(parents)) + n0
    pos_prev = torch.arange(n0)
    allowed = torch.cat([torch.ones(k, n0, dtype=torch.bool), ancestor_mask(parents)], dim=1)
    x = model.w["embed"][torch.tensor(list(z))].to(F64)
    k_new, v_new = [], []
    for l in range(s.n_layers):
        x, k_all, v_all = model._layer(l, x, pos, cache.k[l], cache.v[l], pos_prev, None, allowed)
        k_new.append(k_all[n0:])
        v_new.append(v_all[n0:])
    return model._head(x), k_new, v_new


def accepted_path(z: Sequence[int], parents: Sequence[int], t: Sequence[int]) -> List[int]:
    """SelectLongestAcceptedPrefix on a tree: node indices from the root along matching children."""
    path = [0]
    u = 0
    while True:
        nxt = next((c for c in range(u + 1, len(z)) if parents[c] == u and z[c] == t[u]), None)
        if nxt is None:
            return path
        path.append(nxt)
        u = nxt


def verify_tree(model: OracleModel, pending: int, tokens: Sequence[int], parents: Sequence[int],
                cache: KVCache, want_logits: bool = False):
    """One speculative step over a draft tree.  tokens: draft tokens of nodes 1..k-1; parents: all k
    parents.  The cache grows by the accepted path (root included).  Returns dict(accept_len,
    emitted, argmax, path[, logits])."""
    z = [pending] + list(tokens)
    assert len(z) == len(parents)
    logits, k_new, v_new = forward_tree(model, z, parents, cache)
    t = argmax_lowest(logits)
    path = accepted_path(z, parents, t)
    idx = torch.tensor(path)
    for l in range(model.s.n_layers):
        cache.k[l] = torch.cat([cache.k[l], k_new[l][idx]], dim=0)
        cache.v[l] = torch.cat([cache.v[l], v_new[l][idx]], dim=0)
    res = dict(accept_len=len(path) - 1, emitted=[z[c] for c in path[1:]] + [t[path[-1]]], argmax=t, path=path)
    if want_logits:
        res["logits"] = logits
    return res
