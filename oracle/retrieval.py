"""CPU oracle for the Top-K stage of retrieval (Section 4.3, Eq. 3).

TEST INFRASTRUCTURE ONLY (see oracle/transformer.py).

I_k = Top-K over the datastore of sim(h_i, h_j), sim = cosine similarity between the query's hidden
state and the stored hidden state of each historical invocation.  Ties go to the lower index; a
vector of zero norm has no direction and ranks last (score -2).  The indices, best first, are the
candidate order the suffix match scans.
"""
from typing import List, Tuple

import torch

from .transformer import F64


def cosine_scores(H: torch.Tensor, q: torch.Tensor) -> torch.Tensor:
    """H: [N, d], q: [d] -> [N] float64."""
    H, q = H.to(F64), q.to(F64)
    hn = torch.sqrt((H * H).sum(dim=1))
    qn = torch.sqrt((q * q).sum())
    s = (H @ q) / (hn * qn)
    return torch.where((hn > 0) & (qn > 0), s, torch.full_like(s, -2.0))


def topk_cosine(H: torch.Tensor, q: torch.Tensor, K: int) -> Tuple[List[int], List[float]]:
    s = cosine_scores(H, q)
    order = sorted(range(s.numel()), key=lambda j: (-float(s[j]), j))[:K]
    return order, [float(s[j]) for j in order]


class HiddenStore:
    """The h_j half of the datastore H = {(h_j, y_j)} (Section 4.3): one hidden state per historical invocation, in
    insertion order, the paper's "hidden representation of the input question at its final token".  States are kept
    rounded to bf16, the storage type of the GPU datastore (a reading: the paper does not fix a type); the
    similarity itself is float64."""

    def __init__(self):
        self.rows: List[torch.Tensor] = []

    def add(self, h: torch.Tensor):
        self.rows.append(h.to(torch.bfloat16))

    def retrieve(self, h_x: torch.Tensor, K: int) -> Tuple[List[int], List[float]]:
        """I_k of Eq. 3 for the query state h_x: indices of the K most similar entries, best first (all entries if the
        store holds fewer than K)."""
        return topk_cosine(torch.stack(self.rows), h_x, min(K, len(self.rows)))
