"""GPU parity of the hit-count scores (paper Sec. 5.4 "Aggressive Approximation: hit count-based
Method") against the CPU oracle.  The reported values are small integers and ties are decided by
id on both sides, so values and id lists must be identical, not merely within a tolerance."""

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from conftest import Workload, small_cfg
from ivfpq_inputs import CONFIGS
from test_oracle_pins import _golden, hand_index

pytestmark = pytest.mark.gpu

F32 = np.float32
SCORES = [lib.IVFPQ_SCORE_HIT_COUNT, lib.IVFPQ_SCORE_REWARD_PENALTY]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


def assert_identical(d, i, o):
    assert np.array_equal(host(i), o["ids"])
    assert np.array_equal(host(d).view(np.uint32), o["dist"].view(np.uint32))


def test_hand_worked_scores_on_gpu():
    g = _golden("hand_example.txt")
    nums = lambda k: [float(x) for x in g[k].split()]
    h = lib.ivfpq_index_load(hand_index())
    try:
        q, rad = dev(np.array([nums("query")], F32)), dev(np.array(nums("radius"), F32))
        for score, key in ((lib.IVFPQ_SCORE_HIT_COUNT, "count"), (lib.IVFPQ_SCORE_REWARD_PENALTY, "reward")):
            d, i = lib.ivfpq_search_sparse(h, q, 2, rad, 5, score=score)
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            assert host(i)[0].tolist() == nums(key + "_ids") and host(d)[0].tolist() == nums(key + "_value")
    finally:
        lib.ivfpq_index_free(h)


@pytest.fixture(scope="module")
def shaped():
    out = {}
    for name, base, kw in (
        ("16x8", "c1", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
        ("48x2", "c3", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
        ("50x4", "c4", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
        ("10x3", "c4", dict(n=9_000, d=30, nsub=10, dsub=3, ncomp=100, nlist=37, nq=50)),
    ):
        wl = Workload(small_cfg(base, chunk=16384, kmeans_iters=4, **kw))
        out[name] = (wl, lib.ivfpq_index_load(wl.index))
    yield out
    for _, h in out.values():
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("score", SCORES)
@pytest.mark.parametrize("name", ["16x8", "48x2", "50x4", "10x3"])
def test_scores_identical_to_oracle(shaped, name, score):
    wl, h = shaped[name]
    q = dev(wl.queries)
    for rad, scale, k in ((wl.radius, 1.0, 100), (wl.radius_per_query, 0.6, 100), (wl.radius, 1.7, 1000),
                          (wl.radius, 0.0, 10), (wl.radius, float("inf"), 33)):
        d, i = lib.ivfpq_search_sparse(h, q, 6, dev(rad), k, scale=scale, score=score)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        assert_identical(d, i, oracle.search(wl.index, wl.queries, 6, k, radius=rad, scale=scale, score=score))


@pytest.mark.parametrize("score", SCORES)
@pytest.mark.parametrize("name", ["16x8", "48x2", "50x4", "10x3"])
def test_score_of_every_visited_point(shaped, name, score):
    wl, h = shaped[name]
    nq, nprobe, stride = 24, 5, 6000
    q, rad = wl.queries[:nq], wl.radius_per_query[:nq]
    g = lib.ivfpq_debug_search(h, dev(q), nprobe, 50, radius=dev(rad), scale=1.2, visit_stride=stride, score=score)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    g = {k2: host(v) for k2, v in g.items()}
    o = oracle.search(wl.index, q, nprobe, 50, radius=rad, scale=1.2, dumps=True, visit_stride=stride, score=score)
    assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
    assert np.array_equal(g["visit_count"], o["visit_count"])
    assert np.array_equal(g["visit_ids"], o["visit_ids"])
    assert np.array_equal(g["visit_hits"].view(np.uint64), o["visit_hits"])
    assert np.array_equal(g["visit_dist"].view(np.uint32), o["visit_dist"].view(np.uint32))
    assert len(np.unique(o["visit_dist"][np.isfinite(o["visit_dist"])])) > 3
    assert np.array_equal(g["ids"], o["ids"]) and np.array_equal(g["dist"], o["dist"])


@pytest.mark.parametrize("kernel", ["warps16", "warps32"])
def test_scores_on_both_16x8_kernels_with_splits(kernel, monkeypatch):
    monkeypatch.setenv("IVFPQ_SCAN_KERNEL", kernel)
    wl = Workload(small_cfg("c1", n=40_000, ncomp=300, nlist=160, nq=40, chunk=16384, kmeans_iters=4))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nsplit in (0, 3):
            lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
            for score in SCORES:
                for nprobe, k in ((7, 100), (160, 1000), (1, 10)):
                    d, i = lib.ivfpq_search_sparse(h, q, nprobe, dev(wl.radius), k, scale=0.9, score=score)
                    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
                    assert_identical(d, i, oracle.search(wl.index, wl.queries, nprobe, k, radius=wl.radius,
                                                         scale=0.9, score=score))
    finally:
        lib.ivfpq_index_free(h)


def test_host_entry_point_and_errors(shaped):
    wl, h = shaped["16x8"]
    nq, k = wl.queries.shape[0], 20
    qh = torch.from_numpy(wl.queries).pin_memory()
    od, oi = torch.empty((nq, k), dtype=torch.float32).pin_memory(), torch.empty((nq, k), dtype=torch.int32).pin_memory()
    lib.ivfpq_search_host(h, qh, 4, k, od, oi, radius=dev(wl.radius), score=lib.IVFPQ_SCORE_HIT_COUNT)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    o = oracle.search(wl.index, wl.queries, 4, k, radius=wl.radius, score=1)
    assert np.array_equal(oi.numpy(), o["ids"]) and np.array_equal(od.numpy(), o["dist"])
    for bad in (-1, 3):
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_search_sparse(h, dev(wl.queries), 4, dev(wl.radius), k, score=bad)
        assert e.value.code == lib.IVFPQ_ERR_INVALID_ARGUMENT


@pytest.mark.parametrize("score", SCORES)
def test_full_size_c2_scores_sampled_queries(score):
    """The benchmark's launch configuration (C2, the whole 10 k-query batch, nprobe 16), a sample
    of the queries checked against the oracle, plus properties that hold for every query."""
    wl = Workload(CONFIGS["c2"], device="cuda")
    h = lib.ivfpq_index_load(wl.index)
    try:
        k = wl.cfg.k
        d, i = lib.ivfpq_search_sparse(h, dev(wl.queries), 16, dev(wl.radius), k, scale=0.75, score=score)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        sel = np.sort(np.random.default_rng(1).choice(wl.queries.shape[0], 96, replace=False))
        o = oracle.search(wl.index, wl.queries[sel], 16, k, radius=wl.radius, scale=0.75, score=score)
        gd, gi = host(d), host(i)
        assert np.array_equal(gi[sel], o["ids"]) and np.array_equal(gd[sel], o["dist"])
        assert (np.diff(gd, axis=1) >= 0).all() and (gd == np.round(gd)).all()
        assert gd.min() >= 0 and gd.max() <= wl.index.nsub * score
        tie = gd[:, 1:] == gd[:, :-1]
        assert (gi[:, 1:][tie] > gi[:, :-1][tie]).all()
    finally:
        lib.ivfpq_index_free(h)
