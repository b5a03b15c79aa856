"""GPU parity of the dynamic threshold front-end (paper Sec. 4.1 "Determining Proper Threshold";
Algorithm 2, the threshold step) against the CPU oracle: thresholds are fp32 results of a table look-up and a
fixed-order Horner evaluation, so the comparison is bit for bit."""

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from ivfpq_inputs import ThresholdModel, lossless_toy_index
from parity import assert_topk_parity
from test_threshold_pins import _golden

pytestmark = pytest.mark.gpu

F32 = np.float32


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def random_model(rng, nsub, grid, degree, lo=-1.0, hi=1.0, coef_scale=(0.2, 0.004, -0.00002, 1e-7)):
    dens = (rng.random((nsub, grid, grid)) * 60).astype(F32)
    org = (lo + 0.05 * rng.standard_normal((nsub, 2))).astype(F32)
    inv = (grid / (hi - lo) * (1 + 0.1 * rng.random((nsub, 2)))).astype(F32)
    coef = (np.abs(rng.standard_normal((nsub, degree + 1))) * np.array(coef_scale[:degree + 1])).astype(F32)
    return ThresholdModel(grid, degree, dens, org, inv, coef)


def test_hand_worked_threshold_example_on_gpu():
    g = _golden()
    idx, _ = lossless_toy_index(seed=5, n=64, nlist=4, nsub=1, dsub=2, ksub=16, spread=3.0)
    h = lib.ivfpq_index_load(idx)
    try:
        dens = np.array([[float(x) for x in row.split()] for row in g["density"].split(";")], F32)[None]
        model = ThresholdModel(int(g["grid"]), 1, dens, np.array([[float(x) for x in g["origin"].split()]], F32),
                               np.array([[float(x) for x in g["inv_cell"].split()]], F32),
                               np.array([[float(x) for x in g["coef"].split()]], F32))
        r = lib.ivfpq_query_thresholds(h, dev(np.array(g["query"], F32)), lib.ThresholdModelHandle(model))
        assert r.cpu().numpy().ravel().tolist() == [float(x) for x in g["thresholds"].split()]
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("grid,degree,nq", [(100, 2, 5000), (7, 0, 1), (1, 3, 333), (512, 3, 70001)])
def test_thresholds_bit_equal(wl_pq2, grid, degree, nq):
    wl = wl_pq2
    rng = np.random.default_rng(grid * 10 + degree)
    h = lib.ivfpq_index_load(wl.index)
    try:
        nsub = wl.index.nsub
        q = (rng.random((nq, 2 * nsub)) * 2.6 - 1.3).astype(F32)          # part of them outside the grid
        q[::97, 3] = np.nan                                               # undefined projection: border cell 0
        q[::89, 0] = np.inf
        q[::83, 1] = -np.inf
        model = random_model(rng, nsub, grid, degree)
        model.coef[0, 0] = -5.0                                           # negative values clamp to zero
        want = oracle.thresholds(2 * nsub, nsub, 2, q, model)
        got = lib.ivfpq_query_thresholds(h, dev(q), lib.ThresholdModelHandle(model)).cpu().numpy()
        assert got.shape == want.shape
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
        assert (got[:, 0] == 0).any()
    finally:
        lib.ivfpq_index_free(h)


def test_gpu_thresholds_drive_the_sparse_search(wl_pq2):
    """Front-end + search: thresholds computed on the device feed the sparse search (per-query,
    per-subspace radii), against the oracle's thresholds feeding the oracle's search."""
    wl = wl_pq2
    rng = np.random.default_rng(11)
    h = lib.ivfpq_index_load(wl.index)
    try:
        nsub = wl.index.nsub
        model = random_model(rng, nsub, 100, 2, coef_scale=(0.05, 0.004, -0.00002))
        q = dev(wl.queries)
        rad = lib.ivfpq_query_thresholds(h, q, lib.ThresholdModelHandle(model))
        d, i = lib.ivfpq_search_sparse(h, q, 6, rad, 30)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        orad = oracle.thresholds(2 * nsub, nsub, 2, wl.queries, model)
        assert np.array_equal(rad.cpu().numpy(), orad)
        o = oracle.search(wl.index, wl.queries, 6, 30, radius=orad, dumps=True)
        assert_topk_parity(d.cpu().numpy(), i.cpu().numpy(), o["dist"], o["ids"])
        frac = np.unpackbits(o["masks"].view(np.uint8)).mean() * 256 / wl.index.ksub
        assert 0.02 < frac < 0.98          # the model selects part of every codebook, not all or nothing
    finally:
        lib.ivfpq_index_free(h)


def test_threshold_errors(wl_small, wl_pq2):
    rng = np.random.default_rng(3)
    h4 = lib.ivfpq_index_load(wl_small.index)          # 4-d subspaces: no density map defined
    h2 = lib.ivfpq_index_load(wl_pq2.index)
    try:
        m = lib.ThresholdModelHandle(random_model(rng, wl_small.index.nsub, 10, 1))
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_query_thresholds(h4, dev(wl_small.queries), m)
        assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED
        m = lib.ThresholdModelHandle(random_model(rng, wl_pq2.index.nsub, 10, 1))
        for grid, degree in ((0, 1), (5000, 1), (10, 9), (10, -1)):
            m.struct.grid, m.struct.degree = grid, degree
            with pytest.raises(lib.IvfpqError) as e:
                lib.ivfpq_query_thresholds(h2, dev(wl_pq2.queries), m)
            assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED
        m.struct.grid, m.struct.degree = 10, 1
        m.struct.coef = None
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_query_thresholds(h2, dev(wl_pq2.queries), m)
        assert e.value.code == lib.IVFPQ_ERR_INVALID_ARGUMENT
    finally:
        lib.ivfpq_index_free(h4)
        lib.ivfpq_index_free(h2)


@pytest.mark.parametrize("shape", ["16x8", "50x4", "12x2", "10x3"])
def test_kth_nearest_entry_thresholds_bit_equal(shape):
    """Thresholds from the kth-nearest codebook entry (any subspace width): the CUDA kernel and the
    oracle take the same fp32 steps, so the radii are bit-equal; they then drive the sparse search."""
    from conftest import Workload, small_cfg
    from parity import assert_topk_parity
    cfgs = {"16x8": ("c1", dict(n=12_000, ncomp=120, nlist=40, nq=70)),
            "50x4": ("c4", dict(n=12_000, ncomp=120, nlist=40, nq=70)),
            "12x2": ("c3", dict(n=8_000, d=24, nsub=12, dsub=2, ncomp=100, nlist=30, nq=70)),
            "10x3": ("c4", dict(n=6_000, d=30, nsub=10, dsub=3, ncomp=80, nlist=23, nq=50))}
    base, kw = cfgs[shape]
    wl = Workload(small_cfg(base, chunk=8192, kmeans_iters=3, **kw))
    h = lib.ivfpq_index_load(wl.index)
    try:
        rng = np.random.default_rng(3)
        q = torch.from_numpy(wl.queries).cuda()
        for kth, degree in ((1, 1), (64, 1), (wl.index.ksub, 0), (17, 3)):
            coef = (rng.standard_normal((wl.index.nsub, degree + 1)) * 0.3).astype(np.float32)
            coef[:, 0] += 0.5
            if degree == 1 and kth == 64:
                coef[:] = np.array([0.0, 1.0], np.float32)     # the kth-nearest-entry distance itself
            g = lib.ivfpq_query_thresholds_knn(h, q, kth, torch.from_numpy(coef).cuda())
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            o = oracle.thresholds_knn(wl.index, wl.queries, kth, coef)
            assert np.array_equal(g.cpu().numpy().view(np.uint32), o.view(np.uint32)), (kth, degree)
        # the identity radii at rank 64 feed the sparse search in per-query mode
        ident = torch.tensor([[0.0, 1.0]] * wl.index.nsub, device="cuda")
        d, i = lib.ivfpq_search_sparse(h, q, 5, lib.ivfpq_query_thresholds_knn(h, q, 64, ident), 30, scale=0.9)
        rad = oracle.thresholds_knn(wl.index, wl.queries, 64, np.tile(np.array([[0.0, 1.0]], np.float32), (wl.index.nsub, 1)))
        oo = oracle.search(wl.index, wl.queries, 5, 30, radius=rad, scale=0.9)
        assert_topk_parity(d.cpu().numpy(), i.cpu().numpy(), oo["dist"], oo["ids"])
        with pytest.raises(lib.IvfpqError):
            lib.ivfpq_query_thresholds_knn(h, q, 0, torch.zeros((wl.index.nsub, 2), device="cuda"))
    finally:
        lib.ivfpq_index_free(h)
