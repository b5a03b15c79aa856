"""Pins for the kth-nearest-entry threshold of the CPU oracle (the stand-in for the density map when
subspaces are not 2-d): a hand-worked example, a numpy fp64 restatement, the harness' independent
radius calibration, and the limiting cases.  None of the expected values comes from the oracle."""

import os

import numpy as np
import pytest
import torch

import oracle
from ivfpq_inputs import calibrate_radius, lossless_toy_index
from ivfpq_inputs.index_build import IvfPqIndex

F32 = np.float32


def _golden():
    cents, entries, queries, cases, coef, kth = [], [], [], [], None, None
    with open(os.path.join(os.path.dirname(__file__), "golden", "threshold_knn_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            key, rest = line.split(None, 1)
            vals = [float(x) for x in rest.split()]
            if key == "centroid":
                cents.append(vals)
            elif key == "entry":
                entries.append(vals)
            elif key == "query":
                queries.append(vals)
            elif key == "coef":
                coef = vals
            elif key == "kth":
                kth = int(vals[0])
            elif key == "thresholds":
                cases.append((kth, vals))
    return np.array(cents, F32), np.array(entries, F32), np.array(queries, F32), np.array([coef], F32), cases


def _index(cent, cb):
    nsub, ksub, dsub = cb.shape
    return IvfPqIndex(d=nsub * dsub, nlist=cent.shape[0], nsub=nsub, dsub=dsub, ksub=ksub, ntotal=0,
                      coarse_centroids=cent, codebooks=cb, list_offsets=np.zeros(cent.shape[0] + 1, np.int64),
                      codes=np.zeros((0, nsub), np.uint8), ids=np.zeros(0, np.int32))


def test_hand_worked_kth_nearest_entry_example():
    cent, entries, q, coef, cases = _golden()
    idx = _index(cent, entries[None])
    assert len(cases) == 3
    for kth, want in cases:
        r = oracle.thresholds_knn(idx, q, kth, coef)
        assert np.allclose(r.ravel(), want, rtol=2e-7, atol=0), (kth, r.ravel(), want)


def test_matches_numpy_fp64_restatement():
    rng = np.random.default_rng(4)
    nlist, nsub, dsub, ksub, nq = 13, 5, 3, 40, 60
    cent = (rng.standard_normal((nlist, nsub * dsub)) * 4).astype(F32)
    cb = rng.standard_normal((nsub, ksub, dsub)).astype(F32)
    q = (cent[rng.integers(0, nlist, nq)] + rng.standard_normal((nq, nsub * dsub))).astype(F32)
    coef = rng.standard_normal((nsub, 3)).astype(F32)
    coef[:, 0] += 3.0
    idx = _index(cent, cb)
    q64, c64, cb64 = q.astype(np.float64), cent.astype(np.float64), cb.astype(np.float64)
    near = ((q64[:, None, :] - c64[None]) ** 2).sum(2).argmin(1)
    res = (q64 - c64[near]).reshape(nq, nsub, 1, dsub)
    d2 = ((res - cb64[None]) ** 2).sum(3)                              # [nq][nsub][ksub]
    for kth in (1, 7, ksub):
        v = np.sqrt(np.partition(d2, kth - 1, axis=2)[:, :, kth - 1])
        want = np.maximum(coef[None, :, 0] + coef[None, :, 1] * v + coef[None, :, 2] * v * v, 0.0)
        got = oracle.thresholds_knn(idx, q, kth, coef)
        assert np.allclose(got, want, rtol=2e-5, atol=1e-5)
        assert (got >= 0).all()


def test_identity_polynomial_averages_to_the_harness_calibration():
    """With the coefficients (0, 1) the threshold is the kth-nearest-entry distance; the harness
    calibrates its static radii as sqrt(mean over queries of the 64th smallest squared distance)
    with torch (GEMM-form cluster assignment, kthvalue): an independent computation of the same
    quantity."""
    from conftest import Workload, small_cfg
    wl = Workload(small_cfg("c1", n=6000, d=32, ncomp=60, nlist=16, nsub=8, dsub=4, nq=300, chunk=4096, kmeans_iters=4))
    q = torch.from_numpy(wl.queries)
    want = calibrate_radius(wl.index, q, entry_rank=64)
    ident = np.tile(np.array([[0.0, 1.0]], F32), (wl.index.nsub, 1))
    v = oracle.thresholds_knn(wl.index, wl.queries, 64, ident).astype(np.float64)
    got = np.sqrt((v ** 2).mean(0))
    assert np.allclose(got, want, rtol=1e-4)


def test_limits_lossless_point_constant_and_negative_polynomials():
    idx, base = lossless_toy_index(seed=8, n=500, nlist=6, nsub=4, dsub=5, ksub=32, spread=20.0)
    ident = np.tile(np.array([[0.0, 1.0]], F32), (idx.nsub, 1))
    # a base point sits (up to the rounding of centroid + entry) on one entry of every subspace
    r = oracle.thresholds_knn(idx, base[:50], 1, ident)
    assert (r < 1e-4).all()
    # nesting in kth
    r5, r9 = oracle.thresholds_knn(idx, base[:50], 5, ident), oracle.thresholds_knn(idx, base[:50], 9, ident)
    assert (r5 <= r9).all() and (r <= r5).all()
    const = np.array([[2.5]] * idx.nsub, F32)
    assert (oracle.thresholds_knn(idx, base[:10], 3, const) == 2.5).all()
    neg = np.tile(np.array([[-1.0, -1.0]], F32), (idx.nsub, 1))
    assert (oracle.thresholds_knn(idx, base[:10], 3, neg) == 0.0).all()
    for bad in (0, 33):
        with pytest.raises(ValueError):
            oracle.thresholds_knn(idx, base[:2], bad, ident)
