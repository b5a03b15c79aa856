"""The five synthetic workloads (stand-ins for the paper's SIFT1M, DEEP1M, TTI1M
and SIFT100M/DEEP100M evaluation sets, Sec. 5 "Dataset"; the real files are not
used anywhere in this repository).

`nsub` is the number of PQ subspaces (the paper's D/M), `dsub` the dimension of
one subspace (the paper's M), `ksub` the entries per codebook (the paper's E).
"""

from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n: int                 # base vectors
    d: int                 # dimension
    ncomp: int             # Gaussian-mixture components
    mean_kind: str         # "uniform100" | "unit_sphere" | "normal"
    sigma: float
    clip_nonneg: bool      # clip values at 0 (SIFT-like, non-negative)
    normalize: bool        # L2-normalise every vector (DEEP-like)
    query_mean_shift: float  # in units of sigma, added to every mean coordinate for queries
    nlist: int
    nsub: int
    dsub: int
    nq: int
    nprobes: Tuple[int, ...]
    k: int = 100
    ksub: int = 256
    kmeans_iters: int = 10
    chunk: int = 1_000_000   # streamed generation chunk (base vectors)
    train_n: int = 0         # 0: train on everything; else train on the first train_n vectors
    data_seed: int = 1234
    query_seed: int = 5678
    kmeans_seed: int = 42

    def scaled(self, **kw) -> "WorkloadConfig":
        """A smaller/larger variant of the same recipe (used by tests)."""
        return replace(self, **kw)


CONFIGS = {
    # smoke / SIFT-shaped
    "c1": WorkloadConfig("c1", n=100_000, d=128, ncomp=1_000, mean_kind="uniform100", sigma=8.0,
                         clip_nonneg=True, normalize=False, query_mean_shift=0.0,
                         nlist=256, nsub=16, dsub=8, nq=1_000, nprobes=(8,)),
    # SIFT1M-shaped
    "c2": WorkloadConfig("c2", n=1_000_000, d=128, ncomp=10_000, mean_kind="uniform100", sigma=8.0,
                         clip_nonneg=True, normalize=False, query_mean_shift=0.0,
                         nlist=1024, nsub=16, dsub=8, nq=10_000, nprobes=(8, 16, 32)),
    # DEEP1M-shaped: unit-norm vectors, 2-d subspaces as in the paper's PQ48 study
    "c3": WorkloadConfig("c3", n=1_000_000, d=96, ncomp=10_000, mean_kind="unit_sphere", sigma=0.1,
                         clip_nonneg=False, normalize=True, query_mean_shift=0.0,
                         nlist=1024, nsub=48, dsub=2, nq=10_000, nprobes=(16,)),
    # TTI1M-shaped: queries drawn from a shifted mixture (cross-modal mismatch); L2 here
    "c4": WorkloadConfig("c4", n=1_000_000, d=200, ncomp=10_000, mean_kind="normal", sigma=0.5,
                         clip_nonneg=False, normalize=False, query_mean_shift=0.5,
                         nlist=1024, nsub=50, dsub=4, nq=10_000, nprobes=(32,)),
    # SIFT100M/DEEP100M-shaped: only codes + ids are kept
    "c5": WorkloadConfig("c5", n=100_000_000, d=128, ncomp=100_000, mean_kind="uniform100", sigma=8.0,
                         clip_nonneg=True, normalize=False, query_mean_shift=0.0,
                         nlist=16384, nsub=16, dsub=8, nq=10_000, nprobes=(32,),
                         train_n=2_000_000),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name.lower()]
