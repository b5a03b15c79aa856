"""The sparsity-aware scan through the entry -> points map (Algorithm 1's Map, Sec. 5.3) against
the CPU oracle, and against the code-streaming scan of the same library: same probe lists, masks
and per-point hit sets bit for bit, distances within tolerance, for every score, on short lists
(many clusters per tile), long lists (several chunks per list), empty lists and degenerate radii."""

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from conftest import Workload, small_cfg
from parity import assert_topk_parity, assert_visits_parity

pytestmark = pytest.mark.gpu

F32 = np.float32
MAP, STREAM = lib.IVFPQ_SPARSE_SCAN_MAP, lib.IVFPQ_SPARSE_SCAN_STREAM


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


@pytest.fixture(scope="module")
def short_lists():
    """16 x 8, 30 k points in 96 lists (about 300 points each, some tiles hold 16 clusters)."""
    wl = Workload(small_cfg("c1", n=30_000, ncomp=300, nlist=96, nq=80, chunk=16384, kmeans_iters=4))
    h = lib.ivfpq_index_load(wl.index)
    yield wl, h
    lib.ivfpq_index_free(h)


@pytest.fixture(scope="module")
def long_lists():
    """16 x 8, 60 k points in 5 lists: every list is longer than one 8192-point chunk."""
    wl = Workload(small_cfg("c1", n=60_000, ncomp=100, nlist=5, nq=40, chunk=16384, kmeans_iters=3))
    assert np.diff(wl.index.list_offsets).max() > 2 * 8192
    h = lib.ivfpq_index_load(wl.index)
    yield wl, h
    lib.ivfpq_index_free(h)


def search(h, mode, *a, **kw):
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, mode)
    try:
        return lib.ivfpq_search_sparse(h, *a, **kw)
    finally:
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, lib.IVFPQ_SPARSE_SCAN_AUTO)


@pytest.mark.parametrize("scale", [0.0, 0.3, 0.7, 1.0, 1.6, 3.0])
@pytest.mark.parametrize("fixture", ["short_lists", "long_lists"])
def test_map_scan_matches_oracle_over_radius(fixture, scale, request):
    wl, h = request.getfixturevalue(fixture)
    q = dev(wl.queries)
    nprobe = min(6, wl.index.nlist)
    d, i = search(h, MAP, q, nprobe, dev(wl.radius), 100, scale=scale)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    o = oracle.search(wl.index, wl.queries, nprobe, 100, radius=wl.radius, scale=scale)
    assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
    # and the streaming scan of the same library agrees with it
    d2, i2 = search(h, STREAM, q, nprobe, dev(wl.radius), 100, scale=scale)
    assert_topk_parity(host(d), host(i), host(d2), host(i2))


@pytest.mark.parametrize("penalty", [0.0, 3.5, 2.0 ** 40, float("inf")])
def test_map_scan_explicit_penalties_and_per_query_radii(short_lists, penalty):
    wl, h = short_lists
    d, i = search(h, MAP, dev(wl.queries), 9, dev(wl.radius_per_query), 40, scale=0.8, miss_penalty=penalty)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    o = oracle.search(wl.index, wl.queries, 9, 40, radius=wl.radius_per_query, scale=0.8, miss_penalty=penalty)
    if np.isinf(penalty):
        # points with a miss all report +inf: compare the finite part, then the ids (ascending) of the rest
        gd, gi = host(d), host(i)
        fin = np.isfinite(o["dist"])
        assert np.array_equal(np.isfinite(gd), fin)
        for qi in range(gd.shape[0]):
            n = int(fin[qi].sum())
            assert_topk_parity(gd[qi:qi + 1, :n], gi[qi:qi + 1, :n], o["dist"][qi:qi + 1, :n], o["ids"][qi:qi + 1, :n])
            assert np.array_equal(gi[qi, n:], o["ids"][qi, n:])
    else:
        assert_topk_parity(host(d), host(i), o["dist"], o["ids"])


@pytest.mark.parametrize("score", [lib.IVFPQ_SCORE_HIT_COUNT, lib.IVFPQ_SCORE_REWARD_PENALTY])
@pytest.mark.parametrize("fixture", ["short_lists", "long_lists"])
def test_map_scan_count_scores_identical_to_oracle(fixture, score, request):
    wl, h = request.getfixturevalue(fixture)
    nprobe = min(7, wl.index.nlist)
    for scale in (0.6, 1.2):
        d, i = search(h, MAP, dev(wl.queries), nprobe, dev(wl.radius), 100, scale=scale, score=score)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        o = oracle.search(wl.index, wl.queries, nprobe, 100, radius=wl.radius, scale=scale, score=score)
        assert np.array_equal(host(i), o["ids"])
        assert np.array_equal(host(d), o["dist"])


@pytest.mark.parametrize("fixture", ["short_lists", "long_lists"])
def test_map_scan_stage_dumps_bit_equal(fixture, request):
    """The stage-dump instance of the map kernel: masks and per-point hit sets bit-equal to the
    oracle's, per-point values within tolerance, for every visited point; it also cross-checks the
    number of map entries that reached a point against the point's codes (status word)."""
    wl, h = request.getfixturevalue(fixture)
    nq, nprobe = 12, min(5, wl.index.nlist)
    q, rad = wl.queries[:nq], wl.radius_per_query[:nq]
    stride = int(np.diff(wl.index.list_offsets).max()) * nprobe
    for score in (0, 1, 2):
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, MAP)
        g = lib.ivfpq_debug_search(h, dev(q), nprobe, 50, radius=dev(rad), scale=1.1, visit_stride=stride, score=score)
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, lib.IVFPQ_SPARSE_SCAN_AUTO)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        g = {k2: host(v) for k2, v in g.items()}
        o = oracle.search(wl.index, q, nprobe, 50, radius=rad, scale=1.1, dumps=True, visit_stride=stride, score=score)
        assert np.array_equal(g["probe_ids"], o["probe_ids"])
        assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
        assert 0 < np.unpackbits(o["masks"].view(np.uint8)).mean() < 1
        assert_visits_parity(g, o, wl.index.nsub)
        assert_topk_parity(g["dist"], g["ids"], o["dist"], o["ids"])


def test_map_scan_many_probes_splits_and_large_k(short_lists):
    """More probed clusters than the kernel stages at a time (128) on an index with short and empty
    lists, alone and split over several CTAs per query, k up to the limit."""
    wl = Workload(small_cfg("c1", n=20_000, ncomp=200, nlist=300, nq=24, chunk=16384, kmeans_iters=3))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nsplit in (1, 3):
            lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
            for nprobe, k in ((200, 100), (300, 1024), (129, 7)):
                d, i = search(h, MAP, q, nprobe, dev(wl.radius), k, scale=1.0)
                assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
                o = oracle.search(wl.index, wl.queries, nprobe, k, radius=wl.radius, scale=1.0)
                assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 0)
    finally:
        lib.ivfpq_index_free(h)


def test_map_scan_degenerate_radii(short_lists):
    """Radii for which no fixed-point scale exists (an infinite radius in one subspace, in all of
    them) are evaluated point by point: same answers as the oracle; an infinite radius everywhere
    is the dense search (points with identical codes tie exactly there, and the streaming kernel's
    lane-dependent summation order may break such ties differently in the last bit)."""
    wl, h = short_lists
    q = wl.queries[:24]
    rad = wl.radius.copy() * 0.7
    rad[3] = np.inf
    d, i = search(h, MAP, dev(q), 4, dev(rad), 300, miss_penalty=7.25)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    o = oracle.search(wl.index, q, 4, 300, radius=rad, miss_penalty=7.25)
    assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
    allinf = np.full(wl.index.nsub, np.inf, F32)
    d, i = search(h, MAP, dev(q), 4, dev(allinf), 50)
    dd, di = lib.ivfpq_search_dense(h, dev(q), 4, 50)
    o = oracle.search(wl.index, q, 4, 50, dense=True)
    assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
    assert_topk_parity(host(dd), host(di), host(d), host(i))


def test_map_scan_query_on_a_base_point():
    """Near-exact duplicates: a query that coincides with an encoded point (up to the rounding of
    centroid + entry) has squared distances around 1e-13 in every subspace, far below anything the
    fixed-point sum resolves; the kernel then evaluates the point from its codes and reports the
    oracle's value."""
    from ivfpq_inputs import lossless_toy_index
    idx, base = lossless_toy_index(seed=11, n=4000, nlist=12, nsub=16, dsub=8, ksub=256, spread=6.0)
    h = lib.ivfpq_index_load(idx)
    try:
        rng = np.random.default_rng(5)
        q = base[rng.integers(0, 4000, 32)].copy()
        q[16:] += (rng.standard_normal((16, idx.d)) * 1e-4).astype(F32)    # near-duplicates: tiny sums
        rad = np.full(idx.nsub, 2.5, F32)
        d, i = search(h, MAP, dev(q), 12, dev(rad), 20)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        o = oracle.search(idx, q, 12, 20, radius=rad)
        assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
        assert (host(d)[:16, 0] < 1e-9).all() and (o["dist"][:16, 0] < 1e-9).all()
    finally:
        lib.ivfpq_index_free(h)


def test_map_option_is_refused_without_a_map():
    wl = Workload(small_cfg("c3", n=6_000, d=24, ncomp=100, nlist=24, nsub=12, dsub=2, nq=8, chunk=5000, kmeans_iters=3))
    h = lib.ivfpq_index_load(wl.index)
    try:
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, MAP)
        assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, STREAM)
    finally:
        lib.ivfpq_index_free(h)
