"""GPU parity of the inner-product path (paper Sec. 4.2 "Inner Product Similarity Support") against
the CPU oracle: probe lists, selected-entry masks and hit sets bit-equal; similarities within 1e-4
of the magnitude of the terms that were summed (they have both signs, so the error does not scale
with the result); id lists equal up to swaps among values that close."""

import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from conftest import Workload, small_cfg
from parity import assert_topk_parity, assert_visits_parity
from test_oracle_pins import _golden, hand_index

pytestmark = pytest.mark.gpu

F32 = np.float32


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


def ip_index(index):
    return dataclasses.replace(index, metric=1)


def magnitude(index, queries):
    """Tolerance floor: 1 % of an upper bound of the summed terms, |q| (max |c| + nsub max |e|), so
    that two similarities agree when they differ by less than 1e-6 of that bound (fp32 sums of up
    to nsub + 1 terms of both signs)."""
    qn = np.linalg.norm(queries, axis=1).max()
    return 0.01 * float(qn * (np.linalg.norm(index.coarse_centroids, axis=1).max()
                       + index.nsub * np.linalg.norm(index.codebooks, axis=2).max()))


def check(g_sim, g_ids, o, floor):
    # the comparison rules are written for ascending costs: compare the negated similarities
    assert_topk_parity(-host(g_sim), host(g_ids), -o["dist"], o["ids"], floor=floor)


def test_hand_worked_inner_product_example_on_gpu():
    g = _golden("hand_example.txt")
    nums = lambda k: [float(x) for x in g[k].split()]
    idx = ip_index(hand_index())
    h = lib.ivfpq_index_load(idx)
    try:
        q = dev(np.array([nums("query")], F32))
        pid, pd = lib.ivfpq_debug_probes(h, q, 2)
        assert host(pid)[0].tolist() == nums("ip_probes") and host(pd)[0].tolist() == nums("ip_probe_sim")
        d, i = lib.ivfpq_search_dense(h, q, 2, 5)
        assert host(i)[0].tolist() == nums("ip_dense_ids") and host(d)[0].tolist() == nums("ip_dense_sim")
        r = lib.ivfpq_debug_search(h, q, 2, 5, radius=dev(np.array(nums("radius"), F32)), visit_stride=8)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        assert host(r["ids"])[0].tolist() == nums("ip_sparse_ids") and host(r["dist"])[0].tolist() == nums("ip_sparse_sim")
        m = host(r["masks"]).view(np.uint32)
        assert [int(m[0, 0, s, 0]) for s in range(2)] == [int(x, 2) for x in g["ip_masks"].split()]
        assert host(r["visit_hits"])[0, :5].tolist() == [int(x, 2) for x in g["ip_hitsets"].split()]
        d, i = lib.ivfpq_search_dense(h, q, 1, 4)
        assert host(i)[0].tolist() == [9, 1, -1, -1] and np.isneginf(host(d)[0, 2:]).all()
    finally:
        lib.ivfpq_index_free(h)


SHAPES = [
    ("16x8", "c1", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
    ("48x2", "c3", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
    ("50x4", "c4", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
    ("10x3", "c4", dict(n=9_000, d=30, nsub=10, dsub=3, ncomp=100, nlist=37, nq=50)),
]


@pytest.fixture(scope="module")
def shaped():
    out = {}
    for name, base, kw in SHAPES:
        wl = Workload(small_cfg(base, chunk=16384, kmeans_iters=4, **kw))
        idx = ip_index(wl.index)
        out[name] = (wl, idx, lib.ivfpq_index_load(idx))
    yield out
    for _, _, h in out.values():
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("name", [s[0] for s in SHAPES])
def test_inner_product_search_matches_oracle(shaped, name):
    wl, idx, h = shaped[name]
    q = dev(wl.queries)
    floor = magnitude(idx, wl.queries)
    pid, pd = lib.ivfpq_debug_probes(h, q, 9)
    o = oracle.search(idx, wl.queries, 9, 10, dense=True, dumps=True)
    assert np.array_equal(host(pid), o["probe_ids"])
    assert np.array_equal(host(pd).view(np.uint32), o["probe_d"].view(np.uint32))
    for nsplit in (0, 3):
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
        d, i = lib.ivfpq_search_dense(h, q, 6, 100)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        check(d, i, oracle.search(idx, wl.queries, 6, 100, dense=True), floor)
        for rad, scale, pen, k in ((wl.radius, 1.0, -1.0, 100), (wl.radius_per_query, 1.5, 3.5, 100),
                                   (wl.radius, 2.0, 0.0, 1000), (wl.radius, 0.0, 1.0, 10),
                                   (wl.radius, float("inf"), -1.0, 33)):
            d, i = lib.ivfpq_search_sparse(h, q, 6, dev(rad), k, scale=scale, miss_penalty=pen)
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            check(d, i, oracle.search(idx, wl.queries, 6, k, radius=rad, scale=scale, miss_penalty=pen), floor)
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 0)


@pytest.mark.parametrize("name", [s[0] for s in SHAPES])
def test_inner_product_more_probes_than_one_staged_tile(shaped, name):
    """80 and 96 probed clusters (all of them): the kernels of the conflict-free layouts stage the list
    metadata of 64 clusters at a time and scan a tile's lists as one block sequence; alone and split
    over several CTAs per query, with stage dumps for a few queries."""
    wl, idx, h = shaped[name]
    q = dev(wl.queries)
    floor = magnitude(idx, wl.queries)
    for nsplit in (0, 5):
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
        for nprobe in sorted({min(80, idx.nlist), idx.nlist}):
            d, i = lib.ivfpq_search_sparse(h, q, nprobe, dev(wl.radius), 100, scale=1.5)
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            check(d, i, oracle.search(idx, wl.queries, nprobe, 100, radius=wl.radius, scale=1.5), floor)
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 0)
    nq, nprobe = 6, min(70, idx.nlist)
    stride = int(np.diff(idx.list_offsets).max()) * nprobe
    g = lib.ivfpq_debug_search(h, dev(wl.queries[:nq]), nprobe, 50, radius=dev(wl.radius), scale=1.5, visit_stride=stride)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    g = {k2: host(v) for k2, v in g.items()}
    o = oracle.search(idx, wl.queries[:nq], nprobe, 50, radius=wl.radius, scale=1.5, dumps=True, visit_stride=stride)
    assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
    assert_visits_parity(g, o, idx.nsub, floor=magnitude(idx, wl.queries[:nq]))


@pytest.mark.parametrize("name", [s[0] for s in SHAPES])
def test_inner_product_stage_dumps(shaped, name):
    wl, idx, h = shaped[name]
    nq, nprobe, stride = 24, 5, 6000
    q, rad = wl.queries[:nq], wl.radius_per_query[:nq]
    floor = magnitude(idx, q)
    g = lib.ivfpq_debug_search(h, dev(q), nprobe, 50, radius=dev(rad), scale=1.5, visit_stride=stride)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    g = {k2: host(v) for k2, v in g.items()}
    o = oracle.search(idx, q, nprobe, 50, radius=rad, scale=1.5, dumps=True, visit_stride=stride)
    assert np.array_equal(g["probe_ids"], o["probe_ids"])
    assert np.array_equal(g["probe_d"].view(np.uint32), o["probe_d"].view(np.uint32))
    assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
    assert 0.01 < np.unpackbits(o["masks"].view(np.uint8)).mean() < 0.99
    assert_visits_parity(g, o, idx.nsub, floor=floor)
    assert_topk_parity(-g["dist"], g["ids"], -o["dist"], o["ids"], floor=floor)


def test_inner_product_host_entry_point_and_limits(shaped):
    wl, idx, h = shaped["50x4"]
    nq, k = wl.queries.shape[0], 20
    qh = torch.from_numpy(wl.queries).pin_memory()
    od, oi = torch.empty((nq, k), dtype=torch.float32).pin_memory(), torch.empty((nq, k), dtype=torch.int32).pin_memory()
    lib.ivfpq_search_host(h, qh, 4, k, od, oi, radius=dev(wl.radius), scale=1.5)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    o = oracle.search(idx, wl.queries, 4, k, radius=wl.radius, scale=1.5)
    assert_topk_parity(-od.numpy(), oi.numpy(), -o["dist"], o["ids"], floor=magnitude(idx, wl.queries))
    # the count scores and the static-scratch filtering are defined for L2 only
    with pytest.raises(lib.IvfpqError) as e:
        lib.ivfpq_search_sparse(h, dev(wl.queries), 4, dev(wl.radius), k, score=lib.IVFPQ_SCORE_HIT_COUNT)
    assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED
    with pytest.raises(lib.IvfpqError) as e:
        lib.ivfpq_probe_static(h, dev(wl.queries), 4)
    assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED


def test_inner_product_full_size_c4_sampled_queries():
    """C4's shape and size (1 M points, 50 x 4, 10 k queries, nprobe 32) under the inner product, the
    whole batch in one call; a sample of the queries against the oracle, properties for all."""
    from ivfpq_inputs import CONFIGS
    wl = Workload(CONFIGS["c4"], device="cuda")
    idx = ip_index(wl.index)
    h = lib.ivfpq_index_load(idx)
    try:
        k = wl.cfg.k
        d, i = lib.ivfpq_search_sparse(h, dev(wl.queries), 32, dev(wl.radius), k, scale=1.0)
        dd, di = lib.ivfpq_search_dense(h, dev(wl.queries), 32, k)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        sel = np.sort(np.random.default_rng(3).choice(wl.queries.shape[0], 48, replace=False))
        floor = magnitude(idx, wl.queries)
        o = oracle.search(idx, wl.queries[sel], 32, k, radius=wl.radius, scale=1.0)
        assert_topk_parity(-host(d)[sel], host(i)[sel], -o["dist"], o["ids"], floor=floor)
        o = oracle.search(idx, wl.queries[sel], 32, k, dense=True)
        assert_topk_parity(-host(dd)[sel], host(di)[sel], -o["dist"], o["ids"], floor=floor)
        gi = host(di)
        assert (np.diff(host(dd), axis=1) <= 0).all()
        assert gi.min() >= 0 and gi.max() < idx.ntotal
        assert (np.diff(np.sort(gi, axis=1), axis=1) > 0).all()
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("nlist", [300, 1100, 8500])
def test_inner_product_probe_lists_through_the_tensor_core_proposal(nlist):
    """Filtering by inner product on shapes the tensor-core kernel serves (d a multiple of 4): the
    TF32 products propose, the fused multiply-add chain decides; full rows (300, 1100 clusters) and
    the fused epilogue lists (8500 clusters), mixed-sign inner products, centroids of very different
    norms, duplicated centroids (ties go to the smaller cluster id)."""
    from ivfpq_inputs import lossless_toy_index
    rng = np.random.default_rng(nlist + 1)
    idx, base = lossless_toy_index(seed=4, n=2 * nlist, nlist=nlist, nsub=8, dsub=8, ksub=16, spread=3.0)
    cent = idx.coarse_centroids * rng.uniform(0.1, 30.0, (nlist, 1)).astype(F32)
    cent[1::9] = cent[0:-1:9][: len(cent[1::9])]
    idx.coarse_centroids = np.ascontiguousarray(cent.astype(F32))
    idx = ip_index(idx)
    h = lib.ivfpq_index_load(idx)
    try:
        q = (rng.standard_normal((130, idx.d)) * rng.uniform(0.01, 50.0, (130, 1))).astype(F32)
        for nprobe in (1, 9, 40):
            pid, pd = lib.ivfpq_debug_probes(h, dev(q), nprobe)
            o = oracle.search(idx, q, nprobe, 1, dense=True, dumps=True)
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            assert np.array_equal(host(pid), o["probe_ids"])
            assert np.array_equal(host(pd).view(np.uint32), o["probe_d"].view(np.uint32))
    finally:
        lib.ivfpq_index_free(h)
