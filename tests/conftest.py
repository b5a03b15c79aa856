import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from ivfpq_inputs import CONFIGS, build_index, calibrate_radius  # noqa: E402
from ivfpq_inputs import generators as G  # noqa: E402


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


class Workload:
    """A built index plus queries and calibrated radii, all numpy, on the host."""

    def __init__(self, cfg, device="cpu", nq=None):
        self.cfg = cfg
        self.index, spec = build_index(cfg, device)
        self.queries = G.queries(cfg, spec, nq).cpu().numpy()
        self.radius = calibrate_radius(self.index, G.calibration_queries(cfg, spec, 256))
        rng = np.random.default_rng(7)
        jitter = 1.0 + 0.25 * rng.random((self.queries.shape[0], cfg.nsub), dtype=np.float32)
        self.radius_per_query = (self.radius[None, :] * jitter).astype(np.float32)


def small_cfg(name, **kw):
    return CONFIGS[name].scaled(**kw)


@pytest.fixture(scope="session")
def wl_small():
    """C1's recipe shrunk: 20k points, d=32 as 8x4, 64 lists, 96 queries."""
    cfg = small_cfg("c1", n=20_000, d=32, ncomp=200, nlist=64, nsub=8, dsub=4, nq=96, chunk=8192,
                    kmeans_iters=5)
    return Workload(cfg)


@pytest.fixture(scope="session")
def wl_pq2():
    """C3's recipe shrunk (unit-norm vectors, 2-d subspaces as in the paper): d=24 as 12x2."""
    cfg = small_cfg("c3", n=12_000, d=24, ncomp=150, nlist=48, nsub=12, dsub=2, nq=64, chunk=5000,
                    kmeans_iters=5)
    return Workload(cfg)
