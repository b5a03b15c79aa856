"""Pins for the inner-product path of the CPU oracle (paper Sec. 4.2 "Inner Product Similarity
Support": filtering by inner product, spheres of radius sqrt(R^2 + |e|^2), table value q_s.e)."""

import numpy as np
import pytest

import oracle
from ivfpq_inputs import lossless_toy_index
from test_oracle_pins import _golden, hand_index

F32 = np.float32


def test_hand_worked_inner_product_example():
    g = _golden("hand_example.txt")
    nums = lambda k: [float(x) for x in g[k].split()]
    idx = hand_index()
    q = np.array([nums("query")], F32)
    o = oracle.search(idx, q, 2, 5, dense=True, metric=1, dumps=True)
    assert o["probe_ids"][0].tolist() == nums("ip_probes") and o["probe_d"][0].tolist() == nums("ip_probe_sim")
    assert o["ids"][0].tolist() == nums("ip_dense_ids") and o["dist"][0].tolist() == nums("ip_dense_sim")
    o = oracle.search(idx, q, 2, 5, radius=np.array(nums("radius"), F32), metric=1, dumps=True, visit_stride=8)
    assert o["ids"][0].tolist() == nums("ip_sparse_ids") and o["dist"][0].tolist() == nums("ip_sparse_sim")
    assert [int(o["masks"][0, 0, s, 0]) for s in range(2)] == [int(x, 2) for x in g["ip_masks"].split()]
    assert o["visit_hits"][0, :5].tolist() == [int(x, 2) for x in g["ip_hitsets"].split()]
    one = oracle.search(idx, q, 1, 4, dense=True, metric=1)
    assert one["ids"][0].tolist() == [9, 1, -1, -1] and np.isneginf(one["dist"][0, 2:]).all()


def test_filtering_is_the_largest_inner_products(wl_small):
    idx, q = wl_small.index, wl_small.queries
    o = oracle.search(idx, q, 7, 5, dense=True, metric=1, dumps=True)
    ip = q.astype(np.float64) @ idx.coarse_centroids.astype(np.float64).T
    for i in range(q.shape[0]):
        order = np.argsort(-ip[i], kind="stable")
        gap = np.abs(np.diff(ip[i][order][:8])).min()
        if gap > 1e-3 * np.abs(ip[i]).max():
            assert o["probe_ids"][i].tolist() == order[:7].tolist()
        assert np.allclose(o["probe_d"][i], ip[i][o["probe_ids"][i]], rtol=1e-5, atol=1e-3)
    assert (np.diff(o["probe_d"], axis=1) <= 0).all()


def test_dense_similarity_is_the_inner_product_with_the_reconstruction(wl_small):
    idx, q = wl_small.index, wl_small.queries[:20]
    o = oracle.search(idx, q, 5, 30, dense=True, metric=1, dumps=True)
    pos_of_id = np.empty(idx.ntotal, np.int64)
    pos_of_id[idx.ids] = np.arange(idx.ntotal)
    list_of_pos = np.searchsorted(idx.list_offsets, np.arange(idx.ntotal), side="right") - 1
    for i in range(q.shape[0]):
        for j in range(30):
            x = pos_of_id[o["ids"][i, j]]
            rec = idx.coarse_centroids[list_of_pos[x]].astype(np.float64).copy()
            for s in range(idx.nsub):
                rec[s * idx.dsub:(s + 1) * idx.dsub] += idx.codebooks[s, idx.codes[x, s]]
            want = float(q[i].astype(np.float64) @ rec)
            assert abs(o["dist"][i, j] - want) <= 1e-4 * max(1.0, abs(want), float(np.abs(q[i]).sum()))
    assert (np.diff(o["dist"], axis=1) <= 0).all()


def test_lossless_index_gives_exact_maximum_inner_product_search():
    idx, base = lossless_toy_index(seed=2, n=500, nlist=8, nsub=4, dsub=2, ksub=32, spread=4.0)
    rng = np.random.default_rng(0)
    q = rng.standard_normal((25, idx.d)).astype(F32) * 3
    o = oracle.search(idx, q, idx.nlist, 10, dense=True, metric=1)
    ip = q.astype(np.float64) @ base.astype(np.float64).T
    for i in range(25):
        order = np.lexsort((np.arange(500), -ip[i]))[:10]
        srt = ip[i][order]
        if np.abs(np.diff(srt)).min() > 1e-3:
            assert o["ids"][i].tolist() == order.tolist()
        assert np.allclose(o["dist"][i], srt, rtol=1e-4, atol=1e-3)


@pytest.mark.parametrize("how", ["radius_inf", "scale_inf"])
def test_infinite_radius_equals_dense(wl_small, how):
    idx, q = wl_small.index, wl_small.queries
    dense = oracle.search(idx, q, 6, 50, dense=True, metric=1)
    if how == "radius_inf":
        sp = oracle.search(idx, q, 6, 50, radius=np.full(idx.nsub, np.inf, F32), metric=1, dumps=True)
    else:
        sp = oracle.search(idx, q, 6, 50, radius=wl_small.radius, scale=float("inf"), metric=1, dumps=True)
    assert np.array_equal(sp["ids"], dense["ids"])
    assert np.array_equal(sp["dist"].view(np.uint32), dense["dist"].view(np.uint32))
    assert (sp["masks"] == 0xFFFFFFFF).all()


def test_selection_is_a_threshold_on_the_inner_product(wl_small):
    """|q_s - e|^2 <= R^2 + |e|^2  <=>  q_s.e >= (|q_s|^2 - R^2) / 2: the spheres of radius
    sqrt(R^2 + |e|^2) select exactly the entries whose inner product clears a per-subspace bound
    (checked in fp64 away from the boundary), the same entries for every probed cluster."""
    idx, q = wl_small.index, wl_small.queries[:24]
    rad = wl_small.radius * 3
    o = oracle.search(idx, q, 3, 5, radius=rad, metric=1, dumps=True)
    assert (o["masks"][:, 0] == o["masks"][:, 1]).all() and (o["masks"][:, 0] == o["masks"][:, 2]).all()
    bits = np.unpackbits(o["masks"][:, 0].view(np.uint8), bitorder="little").reshape(24, idx.nsub, 256)
    checked = 0
    for i in range(24):
        for s in range(idx.nsub):
            qs = q[i, s * idx.dsub:(s + 1) * idx.dsub].astype(np.float64)
            ip = idx.codebooks[s].astype(np.float64) @ qs
            bound = (qs @ qs - float(rad[s]) ** 2) / 2
            safe = np.abs(ip - bound) > 1e-4 * (1 + np.abs(ip) + abs(bound))
            assert np.array_equal(bits[i, s][safe], (ip >= bound)[safe].astype(np.uint8))
            checked += int(safe.sum())
    assert checked > 0.99 * 24 * idx.nsub * 256
    assert 0.02 < bits.mean() < 0.98


def test_nesting_and_full_hit_points(wl_small):
    idx, q = wl_small.index, wl_small.queries[:16]
    small = oracle.search(idx, q, 4, 20, radius=wl_small.radius, scale=2.0, metric=1, dumps=True, visit_stride=5000)
    large = oracle.search(idx, q, 4, 20, radius=wl_small.radius, scale=4.0, metric=1, dumps=True, visit_stride=5000)
    dense = oracle.search(idx, q, 4, 20, dense=True, metric=1, dumps=True, visit_stride=5000)
    assert ((small["masks"] & ~large["masks"]) == 0).all()
    full = (1 << idx.nsub) - 1
    n = int(min(dense["visit_count"].min(), 5000))
    for o in (small, large):
        allhit = o["visit_hits"][:, :n] == full
        assert np.array_equal(o["visit_dist"][:, :n][allhit].view(np.uint32),
                              dense["visit_dist"][:, :n][allhit].view(np.uint32))
        # a missed subspace replaces its term by -P: with P = 0 the similarity is the partial sum
    part = oracle.search(idx, q, 4, 20, radius=wl_small.radius, scale=2.0, miss_penalty=0.0, metric=1,
                         visit_stride=5000)
    pen = oracle.search(idx, q, 4, 20, radius=wl_small.radius, scale=2.0, miss_penalty=7.0, metric=1,
                        visit_stride=5000)
    m = idx.nsub - np.array([[bin(int(x)).count("1") for x in row[:n]] for row in part["visit_hits"]])
    assert np.allclose(part["visit_dist"][:, :n] - 7.0 * m, pen["visit_dist"][:, :n], rtol=1e-5, atol=1e-3)
    assert m.max() > 0


def test_count_scores_are_l2_only(wl_small):
    with pytest.raises(ValueError):
        oracle.search(wl_small.index, wl_small.queries[:2], 2, 5, radius=wl_small.radius, metric=1, score=1)
