"""Pins for the Top-K oracle (Eq. 3): torch's own cosine similarity and top-k, closed forms, and the
printed K."""
import os

import torch
import torch.nn.functional as F

import oracle
from oracle.transformer import F64


def test_scores_match_torch_cosine_similarity_and_topk():
    g = torch.Generator().manual_seed(2)
    H = torch.randn(200, 48, generator=g, dtype=F64)
    q = torch.randn(48, generator=g, dtype=F64)
    ref = F.cosine_similarity(H, q[None, :], dim=1, eps=0.0)
    assert torch.allclose(oracle.cosine_scores(H, q), ref, rtol=0, atol=1e-14)
    idx, sc = oracle.topk_cosine(H, q, 10)
    top = torch.topk(ref, 10)
    assert idx == top.indices.tolist()
    assert torch.allclose(torch.tensor(sc, dtype=F64), top.values, rtol=0, atol=1e-14)


def test_closed_forms_and_ties():
    q = torch.tensor([3.0, 0.0, 4.0], dtype=F64)
    H = torch.stack([q * 7, -q, torch.tensor([0.0, 5.0, 0.0], dtype=F64), torch.zeros(3, dtype=F64), q * 0.1])
    s = oracle.cosine_scores(H, q)
    assert torch.allclose(s, torch.tensor([1.0, -1.0, 0.0, -2.0, 1.0], dtype=F64), rtol=0, atol=1e-15)
    idx, _ = oracle.topk_cosine(H, q, 5)
    assert idx == [0, 4, 2, 1, 3]                     # scale does not matter; ties -> lower index; zero vector last
    assert oracle.topk_cosine(H * 3.0, q * 0.5, 5)[0] == idx


def test_hidden_store_retrieval_is_torch_topk_over_the_stored_rows():
    g = torch.Generator().manual_seed(5)
    hs = torch.randn(37, 64, generator=g, dtype=F64)
    store = oracle.HiddenStore()
    for h in hs:
        store.add(h)
    q = hs[20] + 0.05 * torch.randn(64, generator=g, dtype=F64)
    stored = hs.to(torch.bfloat16).to(F64)                       # what the store keeps: bf16-rounded rows
    ref = torch.topk(F.cosine_similarity(stored, q[None, :], dim=1, eps=0.0), 10)
    idx, sc = store.retrieve(q, 10)
    assert idx == ref.indices.tolist() and idx[0] == 20
    assert torch.allclose(torch.tensor(sc, dtype=F64), ref.values, rtol=0, atol=1e-14)
    assert len(store.retrieve(q, 100)[0]) == 37                  # K above the store size: every entry, ranked


def test_printed_k():
    gold = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")
    vals = dict(line.split("#")[0].split("=", 1) for line in open(gold) if "=" in line.split("#")[0])
    assert int(vals["retrieval_top_k "].strip()) == 10
