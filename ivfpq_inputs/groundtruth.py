"""Exact brute-force neighbours on the raw vectors and the recall metrics.

Recall definitions follow the paper's "Metric" paragraph (Sec. 6.1): R1@k counts
the queries whose k retrieved neighbours contain the true nearest neighbour;
recall@k here is the mean fraction of the true k nearest neighbours that were
retrieved (the paper's R100@1000 with both numbers equal to k).
"""

from __future__ import annotations

import numpy as np
import torch


class ExactKnnAccumulator:
    """Running exact top-k (squared L2, or largest inner product with `metric=1`) of a fixed
    query set over base vectors that arrive in chunks.  For the inner product the values kept
    are the negated similarities, so that "smallest first" holds in both cases."""

    def __init__(self, queries: torch.Tensor, k: int, block: int = 131072, metric: int = 0):
        self.q = queries
        self.k = k
        self.metric = metric
        self.block = block
        self.qn = (queries * queries).sum(1)
        nq = queries.shape[0]
        self.best_d = torch.full((nq, k), float("inf"), device=queries.device)
        self.best_i = torch.full((nq, k), -1, dtype=torch.int64, device=queries.device)

    def add(self, first_id: int, x: torch.Tensor) -> None:
        block = max(1024, min(self.block, (1 << 28) // max(1, self.q.shape[0])))
        for lo in range(0, x.shape[0], block):
            xb = x[lo:lo + block]
            if self.metric == 1:
                d = -(self.q @ xb.T)
            else:
                d = self.qn[:, None] - 2.0 * (self.q @ xb.T) + (xb * xb).sum(1)[None, :]
            kk = min(self.k, xb.shape[0])
            dv, di = torch.topk(d, kk, dim=1, largest=False)
            di = di + (first_id + lo)
            alld = torch.cat([self.best_d, dv], 1)
            alli = torch.cat([self.best_i, di], 1)
            sel = torch.topk(alld, self.k, dim=1, largest=False).indices
            self.best_d = torch.gather(alld, 1, sel)
            self.best_i = torch.gather(alli, 1, sel)

    def result(self):
        order = torch.argsort(self.best_d, dim=1, stable=True)
        return (torch.gather(self.best_i, 1, order).cpu().numpy(),
                torch.gather(self.best_d, 1, order).cpu().numpy())


def exact_knn(base: torch.Tensor, queries: torch.Tensor, k: int):
    acc = ExactKnnAccumulator(queries, k)
    acc.add(0, base)
    return acc.result()


def recall_at_k(found_ids: np.ndarray, true_ids: np.ndarray) -> float:
    """Mean over queries of |found ∩ true| / k, k = true_ids.shape[1]."""
    k = true_ids.shape[1]
    hit = 0
    for f, t in zip(found_ids, true_ids):
        hit += len(np.intersect1d(f[f >= 0], t, assume_unique=False))
    return hit / (k * len(true_ids))


def recall_1_at_k(found_ids: np.ndarray, true_ids: np.ndarray) -> float:
    """Fraction of queries whose retrieved set contains the true nearest neighbour."""
    return float(np.mean((found_ids == true_ids[:, :1]).any(axis=1)))
