"""Pins for the dynamic threshold front-end of the CPU oracle (density-map look-up + polynomial
regressor), and for the harness that builds the maps: facts fixed by the paper's definition and by
arithmetic, none of them produced by the oracle itself."""

import os

import numpy as np
import pytest
import torch

import oracle
from ivfpq_inputs import ThresholdModel, containing_thresholds, density_maps, fit_threshold_model, lossless_toy_index

F32 = np.float32


def _golden():
    out = {"query": []}
    with open(os.path.join(os.path.dirname(__file__), "golden", "threshold_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, rest = line.split(None, 1)
                if key == "query":
                    out["query"].append([float(x) for x in rest.split()])
                else:
                    out[key] = rest
    return out


def test_hand_worked_threshold_example():
    g = _golden()
    grid = int(g["grid"])
    dens = np.array([[float(x) for x in row.split()] for row in g["density"].split(";")], F32)[None]
    model = ThresholdModel(grid, 1, dens, np.array([[float(x) for x in g["origin"].split()]], F32),
                           np.array([[float(x) for x in g["inv_cell"].split()]], F32),
                           np.array([[float(x) for x in g["coef"].split()]], F32))
    r = oracle.thresholds(2, 1, 2, np.array(g["query"], F32), model)
    assert r.ravel().tolist() == [float(x) for x in g["thresholds"].split()]


def test_constant_map_or_constant_polynomial_gives_constant_radius():
    rng = np.random.default_rng(0)
    nsub, grid, nq = 5, 7, 200
    q = rng.standard_normal((nq, 2 * nsub)).astype(F32) * 3
    org, inv = -np.ones((nsub, 2), F32) * 4, np.full((nsub, 2), 7 / 8, F32)
    coef = rng.standard_normal((nsub, 4)).astype(F32)
    # polynomial of degree 0: the density does not matter
    m0 = ThresholdModel(grid, 0, rng.random((nsub, grid, grid), dtype=F32), org, inv, np.abs(coef[:, :1]))
    assert np.array_equal(oracle.thresholds(2 * nsub, nsub, 2, q, m0), np.repeat(np.abs(coef[:, :1]).T, nq, 0))
    # constant density: one value per subspace, = the polynomial at that density (fp64 check)
    dens = np.full((nsub, grid, grid), 0.75, F32)
    m3 = ThresholdModel(grid, 3, dens, org, inv, coef)
    r = oracle.thresholds(2 * nsub, nsub, 2, q, m3)
    want = np.maximum(np.polynomial.polynomial.polyval(0.75, coef.astype(np.float64).T), 0.0)
    assert np.allclose(r, np.repeat(want[None, :], nq, 0), rtol=1e-6, atol=1e-6)
    assert (r == r[0]).all()


def test_negative_polynomial_values_clamp_to_zero():
    m = ThresholdModel(1, 1, np.array([[[2.0]]], F32), np.zeros((1, 2), F32), np.ones((1, 2), F32), np.array([[1.0, -3.0]], F32))
    assert oracle.thresholds(2, 1, 2, np.zeros((3, 2), F32), m).ravel().tolist() == [0.0, 0.0, 0.0]


def test_lookup_and_horner_agree_with_numpy_in_fp64():
    rng = np.random.default_rng(1)
    nsub, grid, nq, deg = 6, 100, 500, 2
    q = (rng.random((nq, 2 * nsub)) * 2.4 - 1.2).astype(F32)           # some projections fall outside the grid
    dens = (rng.random((nsub, grid, grid)) * 50).astype(F32)
    org = -np.ones((nsub, 2), F32)
    inv = np.full((nsub, 2), grid / 2.0, F32)
    coef = (rng.standard_normal((nsub, deg + 1)) * [5, 0.1, 0.001]).astype(F32)
    r = oracle.thresholds(2 * nsub, nsub, 2, q, ThresholdModel(grid, deg, dens, org, inv, coef))
    for s in range(nsub):
        t = (q[:, 2 * s:2 * s + 2].astype(np.float64) - org[s]) * inv[s]
        cell = np.clip(np.floor(t), 0, grid - 1).astype(int)
        d = dens[s][cell[:, 1], cell[:, 0]].astype(np.float64)
        want = np.maximum(np.polynomial.polynomial.polyval(d, coef[s].astype(np.float64)), 0)
        # projections within 1e-4 of a cell border may fall on either side in fp32
        frac = t - np.floor(t)
        safe = ((frac > 1e-4) & (frac < 1 - 1e-4)).all(axis=1)
        assert safe.sum() > 0.9 * nq
        assert np.allclose(r[safe, s], want[safe], rtol=1e-5, atol=1e-5)


def test_density_map_is_count_over_area():
    rng = np.random.default_rng(2)
    nsub, grid, n = 3, 10, 20000
    x = torch.from_numpy(rng.random((n, 2 * nsub)).astype(F32) * 4 - 2)
    lo, hi = torch.full((nsub, 2), -2.0), torch.full((nsub, 2), 2.0)
    dens, org, inv = density_maps([x[:7000], x[7000:]], nsub, grid, (lo, hi))
    for s in range(nsub):
        h, _, _ = np.histogram2d(x[:, 2 * s + 1].numpy(), x[:, 2 * s].numpy(), bins=grid, range=[[-2, 2], [-2, 2]])
        assert np.allclose(dens[s], h / (0.4 * 0.4), rtol=1e-5)       # row = second coordinate
    assert np.allclose(org, -2) and np.allclose(inv, 2.5)
    assert abs(dens.sum() * 0.16 - n * nsub) < 1e-3 * n


def test_containing_threshold_and_fit_on_a_lossless_index():
    """With zero quantisation error the containing threshold of a query that *is* a base point and
    whose only neighbour is itself is 0 in every subspace; the fit of a constant is that constant."""
    idx, base = lossless_toy_index(seed=3, n=400, nlist=8, nsub=4, dsub=2, ksub=32, spread=5.0)
    q = torch.from_numpy(base[:50])
    thr = containing_thresholds(idx, q, np.arange(50)[:, None])
    assert np.abs(thr).max() < 1e-4
    dens = np.ones((4, 5, 5), F32)
    model = fit_threshold_model(idx, dens, np.full((4, 2), -50, F32), np.full((4, 2), 0.05, F32), q,
                                np.arange(50)[:, None], degree=0)
    assert np.abs(model.coef).max() < 1e-4 and model.degree == 0


def test_oracle_rejects_other_subspace_widths():
    m = ThresholdModel(1, 0, np.ones((1, 1, 1), F32), np.zeros((1, 2), F32), np.ones((1, 2), F32), np.ones((1, 1), F32))
    with pytest.raises(ValueError):
        oracle.thresholds(3, 1, 3, np.zeros((1, 3), F32), m)
