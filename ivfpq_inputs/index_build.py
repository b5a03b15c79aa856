"""Offline index construction for the synthetic workloads (harness side).

Follows the conventional IVFPQ training the paper starts from (Sec. 2.1
"Inverted File Index", "Product Quantization"; Algorithm 1 up to the codebook
training): Lloyd k-means over the base vectors gives `nlist` coarse centroids
and a label per vector; one codebook of `ksub` entries per subspace is trained
on the residuals `x - centroid[label(x)]` and shared by all lists; a vector's
code in a subspace is the id of the nearest entry to its residual projection.
The ray-tracing scene and the entry->points map of Algorithm 1 are not built:
the search path streams the codes of each inverted list instead.

None of this is timed or compared between implementations: the CPU oracle and
the CUDA library both read the arrays produced here.
"""

from __future__ import annotations

import struct
from dataclasses import dataclass
from typing import Callable, Iterable, Optional

import numpy as np
import torch

from .configs import WorkloadConfig
from . import generators as G

MAGIC = 0x51505649  # "IVPQ"


@dataclass
class IvfPqIndex:
    d: int
    nlist: int
    nsub: int
    dsub: int
    ksub: int
    ntotal: int
    coarse_centroids: np.ndarray   # [nlist, d] float32
    codebooks: np.ndarray          # [nsub, ksub, dsub] float32 (trained on residuals)
    list_offsets: np.ndarray       # [nlist+1] int64 (CSR)
    codes: np.ndarray              # [ntotal, nsub] uint8, list-contiguous
    ids: np.ndarray                # [ntotal] int32, list-contiguous original ids
    metric: int = 0                # 0 = squared L2

    def list_len(self, c: int) -> int:
        return int(self.list_offsets[c + 1] - self.list_offsets[c])


# ----------------------------------------------------------------------------------------------
# k-means helpers (torch, any device)
# ----------------------------------------------------------------------------------------------

def _assign(x: torch.Tensor, cent: torch.Tensor, block: int = 65536) -> torch.Tensor:
    """Index of the nearest centroid for every row of x (GEMM-form distances)."""
    cn = (cent * cent).sum(1)
    out = torch.empty(x.shape[0], dtype=torch.int64, device=x.device)
    # keep the [block, ncent] tile around 1 GiB at most
    block = max(1024, min(block, (1 << 28) // max(1, cent.shape[0])))
    for lo in range(0, x.shape[0], block):
        xb = x[lo:lo + block]
        dist = cn[None, :] - 2.0 * (xb @ cent.T)
        out[lo:lo + block] = dist.argmin(1)
    return out


def kmeans(x: torch.Tensor, k: int, iters: int, seed: int) -> torch.Tensor:
    """Plain Lloyd iterations; seeded random-sample initialisation; an empty
    cluster keeps its previous centroid."""
    n = x.shape[0]
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    if n >= k:
        init = torch.randperm(n, generator=g)[:k].to(x.device)
    else:
        init = torch.randint(0, n, (k,), generator=g).to(x.device)
    cent = x[init].clone()
    for _ in range(iters):
        lab = _assign(x, cent)
        sums = torch.zeros_like(cent)
        sums.index_add_(0, lab, x)
        cnt = torch.bincount(lab, minlength=k).to(x.dtype)
        nz = cnt > 0
        cent[nz] = sums[nz] / cnt[nz, None]
    return cent


def _encode(res: torch.Tensor, codebooks: torch.Tensor) -> torch.Tensor:
    """uint8 codes [n, nsub] of residuals [n, d]."""
    nsub, ksub, dsub = codebooks.shape
    n = res.shape[0]
    codes = torch.empty((n, nsub), dtype=torch.uint8, device=res.device)
    for s in range(nsub):
        codes[:, s] = _assign(res[:, s * dsub:(s + 1) * dsub].contiguous(), codebooks[s]).to(torch.uint8)
    return codes


def _train(cfg: WorkloadConfig, train: torch.Tensor, pq_sample: int = 262144):
    cent = kmeans(train, cfg.nlist, cfg.kmeans_iters, cfg.kmeans_seed)
    lab = _assign(train, cent)
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.kmeans_seed + 1)
    if train.shape[0] > pq_sample:
        sel = torch.randperm(train.shape[0], generator=g)[:pq_sample].to(train.device)
        res = train[sel] - cent[lab[sel]]
    else:
        res = train - cent[lab]
    codebooks = torch.empty((cfg.nsub, cfg.ksub, cfg.dsub), dtype=torch.float32, device=train.device)
    for s in range(cfg.nsub):
        codebooks[s] = kmeans(res[:, s * cfg.dsub:(s + 1) * cfg.dsub].contiguous(), cfg.ksub,
                              cfg.kmeans_iters, cfg.kmeans_seed + 100 + s)
    return cent, codebooks


def _pack_lists(nlist: int, labels: torch.Tensor, codes: torch.Tensor, ids: torch.Tensor):
    order = torch.sort(labels, stable=True).indices
    counts = torch.bincount(labels, minlength=nlist)
    offsets = torch.zeros(nlist + 1, dtype=torch.int64, device=labels.device)
    offsets[1:] = torch.cumsum(counts, 0)
    return offsets, codes[order], ids[order]


# ----------------------------------------------------------------------------------------------
# public builders
# ----------------------------------------------------------------------------------------------

def build_index_streamed(cfg: WorkloadConfig, spec: G.MixtureSpec,
                         on_chunk: Optional[Callable[[int, torch.Tensor], None]] = None) -> IvfPqIndex:
    """Train on the first `train_n` vectors (all of them when train_n == 0), then
    stream the base set chunk by chunk: assign, encode, keep only labels, codes
    and ids.  `on_chunk(first_id, vectors)` is called with every chunk while it is
    alive (used to accumulate exact neighbours in the same pass)."""
    assert cfg.d == cfg.nsub * cfg.dsub
    nch = G.num_chunks(cfg)
    train_n = cfg.train_n if cfg.train_n else cfg.n
    parts, got, c = [], 0, 0
    while got < train_n and c < nch:
        xb = G.base_chunk(cfg, spec, c)
        parts.append(xb[: train_n - got])
        got += parts[-1].shape[0]
        c += 1
    train = parts[0] if len(parts) == 1 else torch.cat(parts)
    del parts
    cent, codebooks = _train(cfg, train)
    del train

    labels, codes, ids = [], [], []
    for c in range(nch):
        xb = G.base_chunk(cfg, spec, c)
        first = c * cfg.chunk
        if on_chunk is not None:
            on_chunk(first, xb)
        lab = _assign(xb, cent)
        xb.sub_(cent[lab])
        codes.append(_encode(xb, codebooks))
        labels.append(lab.to(torch.int32))
        ids.append(torch.arange(first, first + xb.shape[0], dtype=torch.int32, device=xb.device))
        del xb
    labels = torch.cat(labels).to(torch.int64)
    codes = torch.cat(codes)
    ids = torch.cat(ids)
    offsets, codes, ids = _pack_lists(cfg.nlist, labels, codes, ids)
    return IvfPqIndex(d=cfg.d, nlist=cfg.nlist, nsub=cfg.nsub, dsub=cfg.dsub, ksub=cfg.ksub,
                      ntotal=int(codes.shape[0]),
                      coarse_centroids=cent.cpu().numpy(), codebooks=codebooks.cpu().numpy(),
                      list_offsets=offsets.cpu().numpy(), codes=codes.cpu().numpy(),
                      ids=ids.cpu().numpy())


def build_index(cfg: WorkloadConfig, device="cpu",
                on_chunk: Optional[Callable[[int, torch.Tensor], None]] = None):
    """Convenience: mixture + index for a config. Returns (index, mixture spec)."""
    spec = G.make_mixture(cfg, device)
    return build_index_streamed(cfg, spec, on_chunk), spec


def calibrate_radius(index: IvfPqIndex, calib_queries: torch.Tensor, entry_rank: int = 64) -> np.ndarray:
    """Base hit radius per subspace: sqrt of the mean, over calibration queries
    paired with their nearest coarse centroid, of the `entry_rank`-th smallest
    squared distance between the residual projection and the codebook entries.
    With 256 entries and rank 64 about a quarter of the entries fall inside the
    radius at scale 1, the usage the paper reports (Sec. 3.2).  Returns [nsub] fp32."""
    dev = calib_queries.device
    cent = torch.from_numpy(index.coarse_centroids).to(dev)
    cb = torch.from_numpy(index.codebooks).to(dev)
    lab = _assign(calib_queries, cent)
    res = calib_queries - cent[lab]
    rank = min(entry_rank, index.ksub)
    out = np.empty(index.nsub, dtype=np.float32)
    for s in range(index.nsub):
        r = res[:, s * index.dsub:(s + 1) * index.dsub]
        d2 = ((r[:, None, :] - cb[s][None, :, :]) ** 2).sum(2)
        kth = torch.kthvalue(d2, rank, dim=1).values
        out[s] = float(torch.sqrt(kth.mean()))
    return out


def calibrate_radius_ip(index: IvfPqIndex, calib_queries: torch.Tensor, entry_rank: int = 64) -> np.ndarray:
    """Base radius per subspace for the inner-product metric, where entry e is selected when
    |q_s - e|^2 - |e|^2 = |q_s|^2 - 2 q_s.e <= R^2: sqrt of the mean `entry_rank`-th smallest value
    of that expression over calibration queries (0 where the mean is negative: the spheres of
    radius |e| alone already select more than `entry_rank` entries).  Returns [nsub] fp32."""
    dev = calib_queries.device
    cb = torch.from_numpy(index.codebooks).to(dev)
    rank = min(entry_rank, index.ksub)
    out = np.empty(index.nsub, dtype=np.float32)
    for s in range(index.nsub):
        qs = calib_queries[:, s * index.dsub:(s + 1) * index.dsub]
        v = (qs * qs).sum(1)[:, None] - 2.0 * (qs @ cb[s].T)
        kth = torch.kthvalue(v, rank, dim=1).values
        out[s] = float(torch.sqrt(torch.clamp(kth.mean(), min=0.0)))
    return out


def lossless_toy_index(seed: int, n: int, nlist: int, nsub: int, dsub: int, ksub: int = 256,
                       spread: float = 10.0):
    """A tiny index whose base vectors are *exactly* representable: every vector
    is `centroid[label] + concat_s codebook[s][code_s]` evaluated in fp32, so the
    quantisation error is zero and ADC search over all lists must reproduce the
    exact nearest neighbours.  Returns (index, base vectors [n, d] fp32 in
    original-id order)."""
    rng = np.random.default_rng(seed)
    d = nsub * dsub
    cent = (rng.standard_normal((nlist, d)) * spread).astype(np.float32)
    cb = rng.standard_normal((nsub, ksub, dsub)).astype(np.float32)
    labels = rng.integers(0, nlist, n)
    codes = rng.integers(0, ksub, (n, nsub)).astype(np.uint8)
    base = np.empty((n, d), dtype=np.float32)
    for s in range(nsub):
        base[:, s * dsub:(s + 1) * dsub] = cent[labels, s * dsub:(s + 1) * dsub] + cb[s, codes[:, s]]
    order = np.argsort(labels, kind="stable")
    offsets = np.zeros(nlist + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(np.bincount(labels, minlength=nlist))
    idx = IvfPqIndex(d=d, nlist=nlist, nsub=nsub, dsub=dsub, ksub=ksub, ntotal=n,
                     coarse_centroids=cent, codebooks=cb, list_offsets=offsets,
                     codes=np.ascontiguousarray(codes[order]), ids=order.astype(np.int32))
    return idx, base


# ----------------------------------------------------------------------------------------------
# index file: little-endian header {magic, d, nlist, nsub, dsub, ksub, metric, pad, ntotal}
# followed by coarse centroids, codebooks, list offsets, codes, ids
# ----------------------------------------------------------------------------------------------

_HDR = struct.Struct("<8iq")


def save_index(index: IvfPqIndex, path: str) -> None:
    with open(path, "wb") as f:
        f.write(_HDR.pack(MAGIC, index.d, index.nlist, index.nsub, index.dsub, index.ksub,
                          index.metric, 0, index.ntotal))
        for a, t in ((index.coarse_centroids, np.float32), (index.codebooks, np.float32),
                     (index.list_offsets, np.int64), (index.codes, np.uint8), (index.ids, np.int32)):
            np.ascontiguousarray(a, dtype=t).tofile(f)


def load_index(path: str) -> IvfPqIndex:
    with open(path, "rb") as f:
        hdr = f.read(_HDR.size)
        if len(hdr) != _HDR.size:
            raise ValueError("index file: truncated header")
        magic, d, nlist, nsub, dsub, ksub, metric, _pad, ntotal = _HDR.unpack(hdr)
        if magic != MAGIC:
            raise ValueError("index file: bad magic")
        if min(d, nlist, nsub, dsub, ksub) <= 0 or ntotal < 0 or d != nsub * dsub:
            raise ValueError("index file: inconsistent header")

        def rd(count, t):
            a = np.fromfile(f, dtype=t, count=count)
            if a.size != count:
                raise ValueError("index file: truncated array")
            return a

        cent = rd(nlist * d, np.float32).reshape(nlist, d)
        cb = rd(nsub * ksub * dsub, np.float32).reshape(nsub, ksub, dsub)
        off = rd(nlist + 1, np.int64)
        codes = rd(ntotal * nsub, np.uint8).reshape(ntotal, nsub)
        ids = rd(ntotal, np.int32)
    if off[0] != 0 or off[-1] != ntotal or np.any(np.diff(off) < 0):
        raise ValueError("index file: bad list offsets")
    return IvfPqIndex(d=d, nlist=nlist, nsub=nsub, dsub=dsub, ksub=ksub, ntotal=ntotal,
                      coarse_centroids=cent, codebooks=cb, list_offsets=off, codes=codes, ids=ids,
                      metric=metric)
