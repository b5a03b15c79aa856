"""Seeded Gaussian-mixture generators for base vectors and queries.

Everything is drawn with `torch.Generator` objects seeded from
`numpy.random.SeedSequence([seed, stream, chunk])`, so that a chunk of the base
set can be regenerated on its own (the 100M-point workload never exists in
memory as a whole).  Draws made on the CPU and on a CUDA device use different
torch generators and therefore differ; within one device they are reproducible.
The search parity tests never depend on the values themselves: the CPU oracle
and the CUDA library always read the same already-built index arrays.
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from .configs import WorkloadConfig

STREAM_MEANS = 0
STREAM_BASE = 1
STREAM_QUERY = 2
STREAM_CALIB = 3


def _gen(device, seed: int, stream: int, chunk: int = 0) -> torch.Generator:
    state = np.random.SeedSequence([int(seed), int(stream), int(chunk)]).generate_state(1, np.uint64)[0]
    g = torch.Generator(device=device)
    g.manual_seed(int(state) & 0x7FFF_FFFF_FFFF_FFFF)
    return g


@dataclass
class MixtureSpec:
    means: torch.Tensor      # [ncomp, d] fp32
    sigma: float
    clip_nonneg: bool
    normalize: bool


def make_mixture(cfg: WorkloadConfig, device="cpu") -> MixtureSpec:
    g = _gen(device, cfg.data_seed, STREAM_MEANS)
    if cfg.mean_kind == "uniform100":
        means = torch.rand((cfg.ncomp, cfg.d), generator=g, device=device, dtype=torch.float32) * 100.0
    elif cfg.mean_kind == "unit_sphere":
        means = torch.randn((cfg.ncomp, cfg.d), generator=g, device=device, dtype=torch.float32)
        means = means / means.norm(dim=1, keepdim=True).clamp_min(1e-12)
    elif cfg.mean_kind == "normal":
        means = torch.randn((cfg.ncomp, cfg.d), generator=g, device=device, dtype=torch.float32)
    else:
        raise ValueError(cfg.mean_kind)
    return MixtureSpec(means=means, sigma=cfg.sigma, clip_nonneg=cfg.clip_nonneg, normalize=cfg.normalize)


def sample_mixture(spec: MixtureSpec, n: int, seed: int, stream: int, chunk: int = 0,
                   mean_shift: float = 0.0) -> torch.Tensor:
    """n vectors: a uniformly chosen component mean (+ mean_shift*sigma on every
    coordinate) plus isotropic N(0, sigma^2) noise; then clip / normalise."""
    device = spec.means.device
    g = _gen(device, seed, stream, chunk)
    comp = torch.randint(0, spec.means.shape[0], (n,), generator=g, device=device)
    x = torch.randn((n, spec.means.shape[1]), generator=g, device=device, dtype=torch.float32)
    x.mul_(spec.sigma)
    x.add_(spec.means[comp])
    if mean_shift != 0.0:
        x.add_(mean_shift * spec.sigma)
    if spec.clip_nonneg:
        x.clamp_min_(0.0)
    if spec.normalize:
        x.div_(x.norm(dim=1, keepdim=True).clamp_min(1e-12))
    return x


def base_chunk(cfg: WorkloadConfig, spec: MixtureSpec, chunk: int) -> torch.Tensor:
    lo = chunk * cfg.chunk
    n = min(cfg.chunk, cfg.n - lo)
    return sample_mixture(spec, n, cfg.data_seed, STREAM_BASE, chunk)


def num_chunks(cfg: WorkloadConfig) -> int:
    return (cfg.n + cfg.chunk - 1) // cfg.chunk


def queries(cfg: WorkloadConfig, spec: MixtureSpec, nq: int | None = None) -> torch.Tensor:
    return sample_mixture(spec, cfg.nq if nq is None else nq, cfg.query_seed, STREAM_QUERY, 0,
                          mean_shift=cfg.query_mean_shift)


def calibration_queries(cfg: WorkloadConfig, spec: MixtureSpec, n: int = 1000) -> torch.Tensor:
    return sample_mixture(spec, n, cfg.query_seed, STREAM_CALIB, 0, mean_shift=cfg.query_mean_shift)
