"""Pins for the CPU oracle: facts fixed by the paper and by the mathematics, none of
them produced by the oracle itself or by the CUDA path."""

import math

import numpy as np
import pytest
import torch

import oracle
from ivfpq_inputs import exact_knn, lossless_toy_index, recall_at_k
from ivfpq_inputs.index_build import IvfPqIndex

F32 = np.float32


# ---------------------------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------------------------

def reconstruct(index):
    """[ntotal, d] fp64 reconstructed vectors in list order: centroid + concatenated entries."""
    lab = np.repeat(np.arange(index.nlist), np.diff(index.list_offsets))
    rec = index.coarse_centroids[lab].astype(np.float64)
    for s in range(index.nsub):
        rec[:, s * index.dsub:(s + 1) * index.dsub] += index.codebooks[s, index.codes[:, s]].astype(np.float64)
    return rec


def hand_index():
    """A 2-d toy small enough to work by hand: two subspaces of one dimension, two
    lists, four entries per codebook; every number is a small integer, so fp32 is exact."""
    cent = np.array([[0.0, 0.0], [10.0, 10.0]], F32)
    cb = np.array([[[-2.0], [-1.0], [1.0], [2.0]],
                   [[-3.0], [0.0], [1.0], [3.0]]], F32)
    # list 0: points 0..2, list 1: points 3..4 (ids chosen out of order on purpose)
    codes = np.array([[0, 1], [2, 2], [3, 3], [1, 0], [2, 1]], np.uint8)
    ids = np.array([7, 3, 5, 1, 9], np.int32)
    off = np.array([0, 3, 5], np.int64)
    return IvfPqIndex(d=2, nlist=2, nsub=2, dsub=1, ksub=4, ntotal=5, coarse_centroids=cent,
                      codebooks=cb, list_offsets=off, codes=codes, ids=ids)


# ---------------------------------------------------------------------------------------------
# worked example (hand arithmetic)
# ---------------------------------------------------------------------------------------------

def test_hand_worked_example_dense_and_sparse():
    idx = hand_index()
    q = np.array([[1.0, 1.0]], F32)
    # S1: |q-c0|^2 = 2, |q-c1|^2 = 162 -> probes (0, 1)
    pid, pd = oracle.coarse(idx, q, 2)
    assert pid.tolist() == [[0, 1]] and pd.tolist() == [[2.0, 162.0]]
    # list 0: residual (1,1). entries s0: (-2,-1,1,2) -> d2 (9,4,0,1); s1: (-3,0,1,3) -> (16,1,0,4)
    #   id7 codes(0,1): 9+1=10 ; id3 codes(2,2): 0+0=0 ; id5 codes(3,3): 1+4=5
    # list 1: residual (-9,-9). s0 d2: (49,64,100,121); s1 d2: (36,81,100,144)
    #   id1 codes(1,0): 64+36=100 ; id9 codes(2,1): 100+81=181
    dense = oracle.search(idx, q, 2, 5, dense=True)
    assert dense["ids"].tolist() == [[3, 5, 7, 1, 9]]
    assert dense["dist"].tolist() == [[0.0, 5.0, 10.0, 100.0, 181.0]]
    only0 = oracle.search(idx, q, 1, 4, dense=True)
    assert only0["ids"].tolist() == [[3, 5, 7, -1]]
    assert only0["dist"][0, :3].tolist() == [0.0, 5.0, 10.0] and np.isinf(only0["dist"][0, 3])
    # sparse, radius (2, 1): r2 = (4, 1), P = 5.
    #   list 0 selected: s0 {1,2,3} (d2 4,0,1), s1 {1,2} (d2 1,0)
    #     id7 (0,1): s0 miss, s1 hit 1 -> 1 + 1*5 = 6 ; id3 (2,2): 0 ; id5 (3,3): 1 + miss -> 6
    #   list 1: nothing selected -> both points 2 misses -> 10
    sp = oracle.search(idx, q, 2, 5, radius=np.array([2.0, 1.0], F32), dumps=True, visit_stride=8)
    assert sp["dist"].tolist() == [[0.0, 6.0, 6.0, 10.0, 10.0]]
    assert sp["ids"].tolist() == [[3, 5, 7, 1, 9]]          # ties broken by ascending id
    assert sp["masks"][0, 0, 0, 0] == 0b1110 and sp["masks"][0, 0, 1, 0] == 0b0110
    assert sp["masks"][0, 1].sum() == 0
    assert sp["visit_count"].tolist() == [5]
    assert sp["visit_hits"][0, :5].tolist() == [0b10, 0b11, 0b01, 0, 0]
    # explicit penalty
    sp2 = oracle.search(idx, q, 2, 5, radius=np.array([2.0, 1.0], F32), miss_penalty=1000.0)
    assert sp2["dist"].tolist() == [[0.0, 1001.0, 1001.0, 2000.0, 2000.0]]
    # the scaling factor multiplies the threshold: radius (4, 2) at scale 0.5 is the same search
    sp3 = oracle.search(idx, q, 2, 5, radius=np.array([4.0, 2.0], F32), scale=0.5)
    assert sp3["dist"].tolist() == sp["dist"].tolist() and sp3["ids"].tolist() == sp["ids"].tolist()
    # a point exactly on the threshold is selected (d2 == r2)
    sp4 = oracle.search(idx, q, 1, 3, radius=np.array([3.0, 4.0], F32), dumps=True)
    assert sp4["masks"][0, 0, 0, 0] == 0b1111 and sp4["masks"][0, 0, 1, 0] == 0b1111


def _golden(name):
    import os
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, rest = line.split(None, 1)
                out[key] = rest
    return out


def test_golden_hand_example_file():
    """The same hand-worked example read from tests/golden/hand_example.txt (values written by
    hand, with the passages they follow), so the fixture and the in-line arithmetic cannot drift."""
    g = _golden("hand_example.txt")
    nums = lambda k: [float(x) for x in g[k].split()]
    idx = hand_index()
    assert idx.coarse_centroids.ravel().tolist() == [float(x) for x in g["centroids"].replace(";", " ").split()]
    assert idx.codebooks[0].ravel().tolist() == nums("codebook0") and idx.codebooks[1].ravel().tolist() == nums("codebook1")
    q = np.array([nums("query")], F32)
    pid, pd = oracle.coarse(idx, q, 2)
    assert pid[0].tolist() == nums("probes") and pd[0].tolist() == nums("probe_d")
    o = oracle.search(idx, q, 2, 5, dense=True)
    assert o["ids"][0].tolist() == nums("dense_ids") and o["dist"][0].tolist() == nums("dense_dist")
    o = oracle.search(idx, q, 2, 5, radius=np.array(nums("radius"), F32), dumps=True, visit_stride=8)
    assert o["ids"][0].tolist() == nums("sparse_ids") and o["dist"][0].tolist() == nums("sparse_dist")
    assert [int(o["masks"][0, 0, s, 0]) for s in range(2)] == [int(x, 2) for x in g["masks_list0"].split()]
    assert o["visit_hits"][0, :5].tolist() == [int(x, 2) for x in g["hitsets"].split()]


# ---------------------------------------------------------------------------------------------
# P1: radius -> infinity equals dense, bit for bit
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("how", ["radius_inf", "scale_inf", "radius_inf_per_query"])
def test_p1_infinite_radius_equals_dense(wl_small, how):
    idx, q = wl_small.index, wl_small.queries
    dense = oracle.search(idx, q, 6, 50, dense=True)
    if how == "radius_inf":
        sp = oracle.search(idx, q, 6, 50, radius=np.full(idx.nsub, np.inf, F32), dumps=True)
    elif how == "scale_inf":
        sp = oracle.search(idx, q, 6, 50, radius=wl_small.radius, scale=float("inf"), dumps=True)
    else:
        sp = oracle.search(idx, q, 6, 50, radius=np.full((q.shape[0], idx.nsub), np.inf, F32), dumps=True)
    assert np.array_equal(sp["ids"], dense["ids"])
    assert np.array_equal(sp["dist"].view(np.uint32), dense["dist"].view(np.uint32))
    assert (sp["masks"] == 0xFFFFFFFF).all()


# ---------------------------------------------------------------------------------------------
# P2: ADC distance = squared distance to the reconstructed vector (fp64)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("wl_name", ["wl_small", "wl_pq2"])
def test_p2_adc_equals_distance_to_reconstruction(wl_name, request):
    wl = request.getfixturevalue(wl_name)
    idx, q = wl.index, wl.queries[:32]
    res = oracle.search(idx, q, 5, 40, dense=True, dumps=True, visit_stride=4096)
    rec = reconstruct(idx)
    pos_of_id = np.empty(idx.ntotal, np.int64)
    pos_of_id[idx.ids] = np.arange(idx.ntotal)
    for qi in range(q.shape[0]):
        valid = res["ids"][qi] >= 0
        ref = ((rec[pos_of_id[res["ids"][qi][valid]]] - q[qi].astype(np.float64)) ** 2).sum(1)
        np.testing.assert_allclose(res["dist"][qi][valid], ref, rtol=1e-5)
        # and for every visited point, not only the winners
        n = min(int(res["visit_count"][qi]), 4096)
        ref = ((rec[pos_of_id[res["visit_ids"][qi, :n]]] - q[qi].astype(np.float64)) ** 2).sum(1)
        np.testing.assert_allclose(res["visit_dist"][qi, :n], ref, rtol=1e-5)


# ---------------------------------------------------------------------------------------------
# P3: lossless toy index, all lists probed -> exact nearest neighbours
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("nsub,dsub", [(4, 2), (3, 5), (2, 8)])
def test_p3_lossless_index_reproduces_exact_knn(nsub, dsub):
    idx, base = lossless_toy_index(seed=11, n=1500, nlist=7, nsub=nsub, dsub=dsub)
    rng = np.random.default_rng(5)
    q = (base[rng.integers(0, len(base), 40)] + rng.standard_normal((40, idx.d)) * 0.7).astype(F32)
    k = 20
    res = oracle.search(idx, q, idx.nlist, k, dense=True)
    true_ids, true_d = exact_knn(torch.from_numpy(base).double(), torch.from_numpy(q).double(), k)
    np.testing.assert_allclose(res["dist"], true_d, rtol=2e-5, atol=1e-6)
    for qi in range(len(q)):
        if not np.array_equal(res["ids"][qi], true_ids[qi]):
            # only permutations among (near-)equal distances are acceptable
            assert set(res["ids"][qi][:-1]) - set(true_ids[qi]) == set() or \
                np.isclose(true_d[qi][-1], true_d[qi][-2], rtol=1e-5)
            np.testing.assert_allclose(np.sort(res["dist"][qi]), np.sort(true_d[qi]), rtol=2e-5, atol=1e-6)


# ---------------------------------------------------------------------------------------------
# P4: nesting and monotonicity
# ---------------------------------------------------------------------------------------------

def test_p4_probe_lists_are_prefixes_and_sorted(wl_small):
    idx, q = wl_small.index, wl_small.queries
    p4, d4 = oracle.coarse(idx, q, 4)
    p16, d16 = oracle.coarse(idx, q, 16)
    assert np.array_equal(p16[:, :4], p4) and np.array_equal(d16[:, :4], d4)
    assert (np.diff(d16, axis=1) >= 0).all()
    # against a direct fp64 evaluation: same order wherever the fp64 gaps are not tiny
    ref = ((q[:, None, :].astype(np.float64) - idx.coarse_centroids[None].astype(np.float64)) ** 2).sum(2)
    np.testing.assert_allclose(d16, np.sort(ref, axis=1)[:, :16], rtol=1e-5)
    full, _ = oracle.coarse(idx, q, idx.nlist)
    assert (np.sort(full, axis=1) == np.arange(idx.nlist)[None]).all()


def test_p4_masks_and_hitsets_nest_in_radius(wl_small):
    idx, q = wl_small.index, wl_small.queries[:24]
    prev = None
    for scale in (0.0, 0.5, 1.0, 1.5, 3.0, float("inf")):
        r = oracle.search(idx, q, 4, 10, radius=wl_small.radius, scale=scale, dumps=True, visit_stride=3000)
        if prev is not None:
            assert ((prev["masks"] & ~r["masks"]) == 0).all()
            assert ((prev["visit_hits"] & ~r["visit_hits"]) == 0).all()
            assert np.array_equal(prev["visit_ids"], r["visit_ids"])
        prev = r
    assert (prev["masks"] == 0xFFFFFFFF).all()


def test_p4_recall_monotone_in_nprobe_and_radius(wl_small):
    idx, q = wl_small.index, wl_small.queries
    # exact neighbours of the reconstructed vectors would hide PQ error; use raw data
    from ivfpq_inputs import generators as G
    spec = G.make_mixture(wl_small.cfg)
    base = torch.cat([G.base_chunk(wl_small.cfg, spec, c) for c in range(G.num_chunks(wl_small.cfg))])
    true_ids, _ = exact_knn(base, torch.from_numpy(q), 10)
    last_kth = None
    recalls = []
    for nprobe in (1, 2, 4, 8, 16):
        r = oracle.search(idx, q, nprobe, 10, dense=True)
        recalls.append(recall_at_k(r["ids"], true_ids))
        if last_kth is not None:                       # more candidates never worsen the k-th distance
            assert (r["dist"][:, -1] <= last_kth).all()
        last_kth = r["dist"][:, -1]
    assert all(b >= a - 1e-9 for a, b in zip(recalls, recalls[1:])) and recalls[-1] > 0.3 and recalls[-1] >= recalls[0]
    rr = []
    for scale in (0.25, 0.5, 1.0, 2.0, float("inf")):
        r = oracle.search(idx, q, 8, 10, radius=wl_small.radius, scale=scale)
        rr.append(recall_at_k(r["ids"], true_ids))
    assert all(b >= a - 0.02 for a, b in zip(rr, rr[1:])) and rr[-1] >= rr[0]


# ---------------------------------------------------------------------------------------------
# P5: fully-hit points keep their dense distance; the penalty orders by number of misses
# ---------------------------------------------------------------------------------------------

def test_p5_full_hits_equal_dense_and_penalty_orders(wl_small):
    idx, q = wl_small.index, wl_small.queries[:32]
    stride = 3000
    de = oracle.search(idx, q, 4, 10, dense=True, dumps=True, visit_stride=stride)
    sp = oracle.search(idx, q, 4, 10, radius=wl_small.radius_per_query[:32], scale=1.2, dumps=True,
                       visit_stride=stride)
    full = (1 << idx.nsub) - 1
    seen_full = seen_part = 0
    for qi in range(len(q)):
        n = int(sp["visit_count"][qi])
        assert n == de["visit_count"][qi] <= stride
        hits = sp["visit_hits"][qi, :n]
        allhit = hits == full
        assert np.array_equal(sp["visit_dist"][qi, :n][allhit].view(np.uint32),
                              de["visit_dist"][qi, :n][allhit].view(np.uint32))
        r2 = (wl_small.radius_per_query[qi] * F32(1.2)) ** 2
        P = F32(0)
        for v in r2:
            P = F32(P + v)
        if allhit.any() and (~allhit).any():
            assert sp["visit_dist"][qi, :n][allhit].max() <= P * (1 + 1e-6)
            assert sp["visit_dist"][qi, :n][~allhit].min() >= P * (1 - 1e-6)
        # dist = S + m*P with S the sum of the hit terms (bounded by the hit radii)
        m = idx.nsub - np.array([bin(int(h)).count("1") for h in hits])
        assert (sp["visit_dist"][qi, :n] >= m * P * (1 - 1e-6)).all()
        assert (sp["visit_dist"][qi, :n] <= (m * P + r2.sum()) * (1 + 1e-5)).all()
        seen_full += int(allhit.sum())
        seen_part += int((~allhit).sum())
    assert seen_full > 0 and seen_part > 0


def test_p5_mixed_infinite_radius_gives_infinite_penalty(wl_small):
    idx, q = wl_small.index, wl_small.queries[:8]
    rad = wl_small.radius.copy() * 0.5
    rad[0] = np.inf
    r = oracle.search(idx, q, 4, 2000, radius=rad, dumps=True)
    finite = np.isfinite(r["dist"])
    assert ((r["ids"] >= 0) | ~finite).all()
    assert (np.isinf(r["dist"]) & (r["ids"] >= 0)).any()      # missed points: +inf with a valid id


# ---------------------------------------------------------------------------------------------
# P6 / P7: Algorithm 2's ray test and hit distance against the plain compare (2-d subspaces)
# ---------------------------------------------------------------------------------------------

def ray_sphere_first_hit(origin, direction, center, radius):
    """Smallest t >= 0 with |origin + t*direction - center| = radius, or None (fp64)."""
    oc = origin - center
    a = direction @ direction
    b = 2.0 * (oc @ direction)
    c = oc @ oc - radius * radius
    disc = b * b - 4 * a * c
    if disc < 0:
        return None
    t = (-b - math.sqrt(disc)) / (2 * a)
    return t if t >= 0 else None


def test_p6_p7_ray_time_algebra_matches_threshold_compare(wl_pq2):
    """Unit spheres at the entries (z = 2s+1), a ray from the residual projection at
    z = 2s along +z with t_max = 1 - sqrt(1 - (thres*scale)^2): the ray reports a hit
    exactly when the entry is within thres*scale of the projection, and
    R^2 - (1 - t_hit)^2 is the squared distance stored in the table."""
    idx, q = wl_pq2.index, wl_pq2.queries[:6]
    assert idx.dsub == 2
    thres, scale = wl_pq2.radius.astype(np.float64), 0.8
    assert (thres * scale < 1).all()                   # the scene of Algorithm 2 has R = 1
    r = oracle.search(idx, q, 3, 5, radius=wl_pq2.radius, scale=scale, dumps=True)
    rng = np.random.default_rng(0)
    checked = hits = 0
    for qi in range(len(q)):
        for p in range(3):
            c = r["probe_ids"][qi, p]
            for s in rng.choice(idx.nsub, 4, replace=False):
                res = q[qi, 2 * s:2 * s + 2].astype(np.float64) - idx.coarse_centroids[c, 2 * s:2 * s + 2]
                tmax = 1.0 - math.sqrt(1.0 - (thres[s] * scale) ** 2)
                for e in range(idx.ksub):
                    ent = idx.codebooks[s, e].astype(np.float64)
                    d = math.dist(res, ent)
                    if abs(d - thres[s] * scale) < 1e-5 * max(1.0, d):
                        continue                        # boundary: fp32 vs fp64 may differ
                    t = ray_sphere_first_hit(np.array([res[0], res[1], 2.0 * s]), np.array([0.0, 0.0, 1.0]),
                                             np.array([ent[0], ent[1], 2.0 * s + 1.0]), 1.0)
                    ray_hit = t is not None and t <= tmax
                    sel = bool((r["masks"][qi, p, s, e >> 5] >> (e & 31)) & 1)
                    assert ray_hit == sel
                    checked += 1
                    if ray_hit:
                        hits += 1
                        assert abs((1.0 - (1.0 - t) ** 2) - d * d) < 1e-9       # P7
    assert checked > 10000 and 0 < hits < checked


def test_p7_table_value_is_the_hit_distance(wl_pq2):
    """Sum of ray-derived squared hit distances over all subspaces = the dense ADC distance."""
    idx, q = wl_pq2.index, wl_pq2.queries[:3]
    r = oracle.search(idx, q, 1, 3, dense=True, dumps=True)
    pos_of_id = np.empty(idx.ntotal, np.int64)
    pos_of_id[idx.ids] = np.arange(idx.ntotal)
    for qi in range(len(q)):
        c = r["probe_ids"][qi, 0]
        for j in range(3):
            pid = r["ids"][qi, j]
            if pid < 0:
                continue
            code = idx.codes[pos_of_id[pid]]
            total = 0.0
            for s in range(idx.nsub):
                res = q[qi, 2 * s:2 * s + 2].astype(np.float64) - idx.coarse_centroids[c, 2 * s:2 * s + 2]
                ent = idx.codebooks[s, code[s]].astype(np.float64)
                big_r = 4.0                              # any R larger than every distance works
                t = ray_sphere_first_hit(np.array([res[0], res[1], 0.0]), np.array([0.0, 0.0, 1.0]),
                                         np.array([ent[0], ent[1], big_r]), big_r)
                total += big_r ** 2 - (big_r - t) ** 2   # Eq. "mips3" with the ray starting R below the centre
            assert abs(total - r["dist"][qi, j]) <= 2e-5 * max(total, 1e-6)


# ---------------------------------------------------------------------------------------------
# P8: a deliberately naive second implementation (no table at all)
# ---------------------------------------------------------------------------------------------

def naive_sparse_search(idx, q, nprobe, k, radius, scale, miss_penalty):
    out = []
    f = np.float32
    for qv in q:
        dc = []
        for c in range(idx.nlist):
            a = f(0)
            for j in range(idx.d):
                t = f(qv[j] - idx.coarse_centroids[c, j])
                a = f(np.float64(t) * np.float64(t) + np.float64(a))   # one rounding, as fma
            dc.append((a, c))
        probes = [c for _, c in sorted(dc)[:nprobe]]
        r2 = [f(f(radius[s] * f(scale)) * f(radius[s] * f(scale))) for s in range(idx.nsub)]
        if miss_penalty >= 0:
            P = f(miss_penalty)
        else:
            P = f(0)
            for v in r2:
                P = f(P + v)
        cands = []
        for c in probes:
            for x in range(idx.list_offsets[c], idx.list_offsets[c + 1]):
                S, m = f(0), 0
                for s in range(idx.nsub):
                    ent = idx.codebooks[s, idx.codes[x, s]]
                    d2 = f(0)
                    for j in range(idx.dsub):
                        col = s * idx.dsub + j
                        t = f(f(qv[col] - idx.coarse_centroids[c, col]) - ent[j])
                        d2 = f(np.float64(t) * np.float64(t) + np.float64(d2))
                    if d2 <= r2[s]:
                        S = f(S + d2)
                    else:
                        m += 1
                dist = S if m == 0 else f(np.float64(f(m)) * np.float64(P) + np.float64(S))
                cands.append((dist, int(idx.ids[x])))
        cands.sort()
        out.append(cands[:k])
    return out


@pytest.mark.parametrize("nsub,dsub,penalty", [(4, 2, -1.0), (3, 3, 50.0), (2, 1, -1.0)])
def test_p8_naive_reimplementation_agrees(nsub, dsub, penalty):
    idx, base = lossless_toy_index(seed=3, n=600, nlist=5, nsub=nsub, dsub=dsub, ksub=16, spread=2.0)
    rng = np.random.default_rng(9)
    q = (base[rng.integers(0, 600, 6)] + rng.standard_normal((6, idx.d)) * 0.5).astype(F32)
    radius = np.full(nsub, 1.3, F32)
    ref = naive_sparse_search(idx, q, 3, 25, radius, 0.9, penalty)
    got = oracle.search(idx, q, 3, 25, radius=radius, scale=0.9, miss_penalty=penalty)
    for qi, cands in enumerate(ref):
        assert [i for _, i in cands] == got["ids"][qi, :len(cands)].tolist()
        assert np.array_equal(np.array([d for d, _ in cands], F32).view(np.uint32),
                              got["dist"][qi, :len(cands)].view(np.uint32))
    dense_ref = naive_sparse_search(idx, q, 3, 25, np.full(nsub, np.inf, F32), 1.0, -1.0)
    dense = oracle.search(idx, q, 3, 25, dense=True)
    for qi, cands in enumerate(dense_ref):
        assert [i for _, i in cands] == dense["ids"][qi, :len(cands)].tolist()


# ---------------------------------------------------------------------------------------------
# P9: bookkeeping
# ---------------------------------------------------------------------------------------------

def test_p9_counts_padding_and_zero_radius(wl_small):
    idx, q = wl_small.index, wl_small.queries[:16]
    r = oracle.search(idx, q, 3, 10, radius=wl_small.radius, dumps=True, visit_stride=16)
    lens = np.diff(idx.list_offsets)
    assert np.array_equal(r["visit_count"], lens[r["probe_ids"]].sum(1))
    pop = np.unpackbits(r["masks"].view(np.uint8), axis=-1).reshape(*r["masks"].shape[:3], -1).sum(-1)
    assert (pop <= idx.ksub).all() and 0 < pop.mean() < idx.ksub
    # radius 0: every subspace misses, every distance is nsub * P
    z = oracle.search(idx, q, 3, 10, radius=np.zeros(idx.nsub, F32), miss_penalty=2.5, dumps=True)
    assert (z["masks"] == 0).all()
    assert (z["dist"][z["ids"] >= 0] == F32(idx.nsub * 2.5)).all()
    # fewer candidates than k: padded with (+inf, -1), the rest ascending
    big = oracle.search(idx, q, 1, int(lens.max()) + 5, dense=True)
    for qi in range(len(q)):
        n = lens[r["probe_ids"][qi, 0]]
        assert (big["ids"][qi, n:] == -1).all() and np.isinf(big["dist"][qi, n:]).all()
        assert (big["ids"][qi, :n] >= 0).all() and (np.diff(big["dist"][qi, :n]) >= 0).all()
        assert sorted(big["ids"][qi, :n].tolist()) == sorted(
            idx.ids[idx.list_offsets[r["probe_ids"][qi, 0]]:idx.list_offsets[r["probe_ids"][qi, 0] + 1]].tolist())


def test_oracle_rejects_bad_arguments(wl_small):
    idx, q = wl_small.index, wl_small.queries[:2]
    with pytest.raises(ValueError):
        oracle.search(idx, q, idx.nlist + 1, 5, dense=True)
    with pytest.raises(ValueError):
        oracle.search(idx, q, 2, 5)                      # sparse without radius
    with pytest.raises(ValueError):
        oracle.search(idx, q, 2, 5, radius=np.ones(idx.nsub + 1, F32))
