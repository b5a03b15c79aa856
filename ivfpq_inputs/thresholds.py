"""Offline side of the dynamic threshold (paper Sec. 4.1 "Determining Proper Threshold"): the
per-subspace density maps and the polynomial regressor.  Harness code: it prepares the model that
the search-time front-end (CPU oracle / CUDA library) consumes, and contains none of that front-end.

Density map: every 2-d subspace is divided into a grid x grid map over the bounding box of the
base projections; a cell's density is the number of base projections in it divided by its area.
Regressor: for sampled queries with known exact neighbours, the threshold that contains the entries
of all top-k neighbours in a subspace (the largest distance between the query's residual projection
and the codebook entry of a neighbour) is regressed on the density of the query's cell with a
low-degree polynomial, one per subspace.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Iterable, Tuple

import numpy as np
import torch


@dataclass
class ThresholdModel:
    grid: int
    degree: int
    density: np.ndarray    # [nsub, grid, grid] fp32, row = second coordinate, column = first
    origin: np.ndarray     # [nsub, 2] fp32
    inv_cell: np.ndarray   # [nsub, 2] fp32
    coef: np.ndarray       # [nsub, degree + 1] fp32, ascending powers


def cell_index(x: torch.Tensor, origin: torch.Tensor, inv_cell: torch.Tensor, grid: int) -> torch.Tensor:
    """Grid cell per coordinate, same rule as the search-time look-up (floor, clamped to the border)."""
    t = torch.floor((x - origin) * inv_cell)
    return torch.nan_to_num(t, nan=0.0).clamp_(0, grid - 1).to(torch.int64)


class DensityAccumulator:
    """Density maps of base vectors that arrive in chunks: `add(x)` per chunk [n, 2 * nsub],
    `result()` = (density [nsub, grid, grid], origin [nsub, 2], inv_cell [nsub, 2]) as fp32 numpy.
    extent: (lo [nsub, 2], hi [nsub, 2]) tensors on the device the counting runs on."""

    def __init__(self, nsub: int, grid: int, extent: Tuple[torch.Tensor, torch.Tensor]):
        self.lo, hi = extent
        self.nsub, self.grid = nsub, grid
        cell = (hi - self.lo) / grid
        self.cell = torch.where(cell > 0, cell, torch.ones_like(cell))
        self.inv = (1.0 / self.cell).to(torch.float32)
        self.counts = torch.zeros((nsub, grid * grid), dtype=torch.float64, device=self.lo.device)

    def add(self, x: torch.Tensor) -> None:
        x = x.to(self.lo.device)
        for s in range(self.nsub):
            idx = cell_index(x[:, 2 * s:2 * s + 2], self.lo[s], self.inv[s], self.grid)
            flat = idx[:, 1] * self.grid + idx[:, 0]
            self.counts[s] += torch.bincount(flat, minlength=self.grid * self.grid).to(torch.float64)

    def result(self):
        area = (self.cell[:, 0] * self.cell[:, 1]).to(torch.float64)
        dens = (self.counts / area[:, None]).reshape(self.nsub, self.grid, self.grid).to(torch.float32)
        return dens.cpu().numpy(), self.lo.to(torch.float32).cpu().numpy(), self.inv.cpu().numpy()


def density_maps(chunks: Iterable[torch.Tensor], nsub: int, grid: int,
                 extent: Tuple[torch.Tensor, torch.Tensor]):
    """chunks: base vectors [n, 2 * nsub] (any device); extent: (lo [nsub, 2], hi [nsub, 2]).
    Returns (density [nsub, grid, grid], origin [nsub, 2], inv_cell [nsub, 2]) as fp32 numpy."""
    acc = DensityAccumulator(nsub, grid, extent)
    for x in chunks:
        acc.add(x)
    return acc.result()


def containing_thresholds(index, queries: torch.Tensor, neighbour_ids: np.ndarray) -> np.ndarray:
    """[nq, nsub]: for every query and subspace, the largest distance between the query's residual
    projection (against the centroid of the neighbour's list) and the neighbour's codebook entry,
    over the query's exact neighbours `neighbour_ids` [nq, k] (original ids)."""
    dev = queries.device
    nsub, dsub = index.nsub, index.dsub
    pos_of_id = np.empty(index.ntotal, np.int64)
    pos_of_id[index.ids] = np.arange(index.ntotal)
    list_of_pos = np.repeat(np.arange(index.nlist), np.diff(index.list_offsets))
    pos = pos_of_id[neighbour_ids]                                   # [nq, k]
    cent = torch.from_numpy(index.coarse_centroids).to(dev)
    cb = torch.from_numpy(index.codebooks).to(dev)
    codes = torch.from_numpy(index.codes[pos.ravel()].astype(np.int64)).to(dev).reshape(*pos.shape, nsub)
    lists = torch.from_numpy(list_of_pos[pos]).to(dev)               # [nq, k]
    res = queries[:, None, :] - cent[lists]                          # [nq, k, d]
    out = torch.empty((queries.shape[0], nsub), device=dev)
    for s in range(nsub):
        ent = cb[s][codes[:, :, s]]                                  # [nq, k, dsub]
        dist = (res[:, :, s * dsub:(s + 1) * dsub] - ent).norm(dim=2)
        out[:, s] = dist.max(dim=1).values
    return out.cpu().numpy()


def fit_threshold_model(index, density, origin, inv_cell, queries: torch.Tensor,
                        neighbour_ids: np.ndarray, degree: int = 2) -> ThresholdModel:
    """Least-squares polynomial per subspace: containing threshold as a function of cell density."""
    grid = density.shape[1]
    thr = containing_thresholds(index, queries, neighbour_ids)
    q = queries.cpu()
    coef = np.zeros((index.nsub, degree + 1), np.float32)
    for s in range(index.nsub):
        idx = cell_index(q[:, 2 * s:2 * s + 2], torch.from_numpy(origin[s]), torch.from_numpy(inv_cell[s]), grid).numpy()
        dens = density[s][idx[:, 1], idx[:, 0]].astype(np.float64)
        scale = max(float(dens.max()), 1e-30)                        # condition the fit
        c = np.polynomial.polynomial.polyfit(dens / scale, thr[:, s].astype(np.float64), degree)
        coef[s] = (c / scale ** np.arange(degree + 1)).astype(np.float32)
    return ThresholdModel(grid=grid, degree=degree, density=density.astype(np.float32), origin=origin.astype(np.float32),
                          inv_cell=inv_cell.astype(np.float32), coef=coef)
