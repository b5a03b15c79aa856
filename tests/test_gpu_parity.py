"""Parity of the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from ivfpq_inputs import lossless_toy_index
from conftest import Workload, small_cfg
from parity import assert_topk_parity, assert_visits_parity
from test_oracle_pins import hand_index

pytestmark = pytest.mark.gpu

F32 = np.float32


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


@pytest.fixture(scope="module")
def loaded(wl_small, wl_pq2):
    out = {}
    for name, wl in (("small", wl_small), ("pq2", wl_pq2)):
        out[name] = (wl, lib.ivfpq_index_load(wl.index))
    yield out
    for _, h in out.values():
        lib.ivfpq_index_free(h)


@pytest.fixture(scope="module")
def shaped():
    """Small instances of the three benchmark code shapes (16x8, 48x2, 50x4), so that the
    specialised kernels are the ones under test, plus an odd generic shape (10x3)."""
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


def check_status(h):
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK


# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["small", "pq2"])
@pytest.mark.parametrize("nprobe", [1, 7, 32])
def test_probe_lists_bit_equal(loaded, name, nprobe):
    wl, h = loaded[name]
    pid, pd = lib.ivfpq_debug_probes(h, dev(wl.queries), nprobe)
    opid, opd = oracle.coarse(wl.index, wl.queries, nprobe)
    check_status(h)
    assert np.array_equal(host(pid), opid)
    assert np.array_equal(host(pd).view(np.uint32), opd.view(np.uint32))


def test_probe_lists_tensor_core_shapes():
    """Filtering through the tensor-core proposal + exact decision on shapes that exercise the
    tile edges: d = 200 (seven 32-float K blocks, the last one zero-filled beyond the row),
    nlist = 300 (three centroid tiles, the last one partly outside), 300 queries (three query tiles)."""
    wl = Workload(small_cfg("c4", n=30_000, ncomp=300, nlist=300, nq=300, chunk=16384, kmeans_iters=3))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nprobe in (1, 9, 64, 300):
            pid, pd = lib.ivfpq_debug_probes(h, q, nprobe)
            opid, opd = oracle.coarse(wl.index, wl.queries, nprobe)
            check_status(h)
            assert np.array_equal(host(pid), opid)
            assert np.array_equal(host(pd).view(np.uint32), opd.view(np.uint32))
        # rows that are not 16-byte aligned take the plain kernels: same answer
        q_off = torch.empty(wl.queries.size + 1, dtype=torch.float32, device="cuda")[1:].view(wl.queries.shape)
        q_off.copy_(q)
        pid2, pd2 = lib.ivfpq_debug_probes(h, q_off, 9)
        pid, pd = lib.ivfpq_debug_probes(h, q, 9)
        assert torch.equal(pid, pid2) and torch.equal(pd.view(torch.int32), pd2.view(torch.int32))
    finally:
        lib.ivfpq_index_free(h)


def test_probe_lists_many_clusters():
    """More clusters than the exact decision's candidate buffer holds (the row of approximate
    distances is streamed through it in batches), small and large probe counts."""
    wl = Workload(small_cfg("c1", n=24_000, d=64, nsub=8, dsub=8, ncomp=400, nlist=5000, nq=150, chunk=16384,
                            kmeans_iters=2))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nprobe in (1, 32, 300, 1024):
            pid, pd = lib.ivfpq_debug_probes(h, q, nprobe)
            opid, opd = oracle.coarse(wl.index, wl.queries, nprobe)
            check_status(h)
            assert np.array_equal(host(pid), opid)
            assert np.array_equal(host(pd).view(np.uint32), opd.view(np.uint32))
    finally:
        lib.ivfpq_index_free(h)


def test_probe_lists_fused_selection_large_nlist():
    """8192 clusters or more with few probes: the filtering epilogue keeps only the values under a cut
    taken from the first quarter of the clusters instead of writing full rows; many probes go through
    the full rows.  Same probe lists, bit for bit, either way, also for batches of one and three
    queries (their scratch is chunked differently)."""
    wl = Workload(small_cfg("c1", n=40_000, d=64, nsub=8, dsub=8, ncomp=500, nlist=9000, nq=301, chunk=16384,
                            kmeans_iters=2))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nprobe in (1, 7, 32, 64, 65, 200):
            pid, pd = lib.ivfpq_debug_probes(h, q, nprobe)
            opid, opd = oracle.coarse(wl.index, wl.queries, nprobe)
            check_status(h)
            assert np.array_equal(host(pid), opid)
            assert np.array_equal(host(pd).view(np.uint32), opd.view(np.uint32))
            for n in (1, 3):
                pid, pd = lib.ivfpq_debug_probes(h, q[:n].contiguous(), nprobe)
                check_status(h)
                assert np.array_equal(host(pid), opid[:n])
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("nlist,d", [(300, 64), (1000, 64), (1100, 64), (8500, 64), (1000, 256), (1100, 256)])
def test_probe_lists_large_norms_and_near_ties(nlist, d):
    """Aimed at the error bound of the tensor-core proposal: coordinates around 1e4 with unit spread
    (the TF32 products are off by far more than the distances differ, so nearly every cluster falls
    under the cut), duplicated centroids (exact ties, decided by cluster id) and queries much shorter
    than the centroids, also at the largest dimension the tensor-core path takes (256: the fp32 term of the
    bound grows with d).  A loose bound would drop a true probe; the lists must stay bit-equal."""
    rng = np.random.default_rng(nlist)
    idx, base = lossless_toy_index(seed=9, n=2 * nlist, nlist=nlist, nsub=d // 8, dsub=8, ksub=16, spread=1.0)
    cent = (idx.coarse_centroids + 1.0e4).astype(F32)
    cent[1::7] = cent[0:-1:7][: len(cent[1::7])]           # duplicates: exact ties
    idx.coarse_centroids = cent
    h = lib.ivfpq_index_load(idx)
    try:
        q_far = (cent[rng.integers(0, nlist, 96)] + rng.standard_normal((96, d))).astype(F32)
        q_short = (rng.standard_normal((32, d)) * 1.0e2).astype(F32)      # |q| about 1e-2 of |c|
        q = np.concatenate([q_far, q_short])
        for nprobe in (1, 8, 33):
            pid, pd = lib.ivfpq_debug_probes(h, dev(q), nprobe)
            opid, opd = oracle.coarse(idx, q, nprobe)
            check_status(h)
            assert np.array_equal(host(pid), opid)
            assert np.array_equal(host(pd).view(np.uint32), opd.view(np.uint32))
    finally:
        lib.ivfpq_index_free(h)


def test_probe_all_lists(loaded):
    wl, h = loaded["small"]
    pid, pd = lib.ivfpq_debug_probes(h, dev(wl.queries), wl.index.nlist)
    opid, opd = oracle.coarse(wl.index, wl.queries, wl.index.nlist)
    assert np.array_equal(host(pid), opid)
    assert np.array_equal(host(pd).view(np.uint32), opd.view(np.uint32))


@pytest.mark.parametrize("name", ["small", "pq2"])
@pytest.mark.parametrize("nprobe,k", [(4, 10), (9, 100), (3, 1)])
def test_dense_search_matches_oracle(loaded, name, nprobe, k):
    wl, h = loaded[name]
    d, i = lib.ivfpq_search_dense(h, dev(wl.queries), nprobe, k)
    check_status(h)
    o = oracle.search(wl.index, wl.queries, nprobe, k, dense=True)
    assert_topk_parity(host(d), host(i), o["dist"], o["ids"])


@pytest.mark.parametrize("name", ["16x8", "48x2", "50x4", "10x3"])
def test_benchmark_code_shapes_dense_and_sparse(shaped, name):
    wl, h = shaped[name]
    q = dev(wl.queries)
    d, i = lib.ivfpq_search_dense(h, q, 6, 100)
    o = oracle.search(wl.index, wl.queries, 6, 100, dense=True)
    check_status(h)
    assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
    for scale in (0.7, 1.0, 1.6):
        d, i = lib.ivfpq_search_sparse(h, q, 6, dev(wl.radius), 100, scale=scale)
        o = oracle.search(wl.index, wl.queries, 6, 100, radius=wl.radius, scale=scale)
        check_status(h)
        assert_topk_parity(host(d), host(i), o["dist"], o["ids"])


@pytest.mark.parametrize("name", ["16x8", "48x2", "50x4", "10x3"])
def test_stage_dumps_bit_equal(shaped, name):
    """Probe lists, selected-entry masks and per-point hit sets are bit-equal; per-point
    distances within tolerance; for every visited point, not only the winners."""
    wl, h = shaped[name]
    nq, nprobe, stride = 24, 5, 6000
    q = wl.queries[:nq]
    rad = wl.radius_per_query[:nq]
    g = lib.ivfpq_debug_search(h, dev(q), nprobe, 50, radius=dev(rad), scale=1.1, visit_stride=stride)
    check_status(h)
    g = {k2: host(v) for k2, v in g.items()}
    o = oracle.search(wl.index, q, nprobe, 50, radius=rad, scale=1.1, dumps=True, visit_stride=stride)
    assert np.array_equal(g["probe_ids"], o["probe_ids"])
    assert np.array_equal(g["probe_d"].view(np.uint32), o["probe_d"].view(np.uint32))
    assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
    assert 0 < np.unpackbits(o["masks"].view(np.uint8)).mean() < 1
    assert_visits_parity(g, o, wl.index.nsub)
    assert_topk_parity(g["dist"], g["ids"], o["dist"], o["ids"])
    # dense dumps: every mask bit set, distances follow the same summation order as the oracle
    g = lib.ivfpq_debug_search(h, dev(q), nprobe, 50, visit_stride=stride)
    g = {k2: host(v) for k2, v in g.items()}
    o = oracle.search(wl.index, q, nprobe, 50, dense=True, dumps=True, visit_stride=stride)
    assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
    assert_visits_parity(g, o, wl.index.nsub)


@pytest.mark.parametrize("kernel", ["warps16", "warps32"])
def test_16x8_kernels_forced(kernel, monkeypatch):
    """The 16 x 8 shape has two kernels, chosen by mean list length when the index is loaded;
    force each of them on the same small index: top-k parity (dense, sparse) and stage dumps."""
    monkeypatch.setenv("IVFPQ_SCAN_KERNEL", kernel)
    wl = Workload(small_cfg("c1", n=40_000, ncomp=300, nlist=64, nq=70, chunk=16384, kmeans_iters=4))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nprobe, k in ((7, 100), (64, 1000), (1, 10)):
            d, i = lib.ivfpq_search_dense(h, q, nprobe, k)
            o = oracle.search(wl.index, wl.queries, nprobe, k, dense=True)
            check_status(h)
            assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
            d, i = lib.ivfpq_search_sparse(h, q, nprobe, dev(wl.radius_per_query), k, scale=0.9)
            o = oracle.search(wl.index, wl.queries, nprobe, k, radius=wl.radius_per_query, scale=0.9)
            check_status(h)
            assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
        nq, nprobe, stride = 16, 5, 8000
        qs, rad = wl.queries[:nq], wl.radius_per_query[:nq]
        g = lib.ivfpq_debug_search(h, dev(qs), nprobe, 50, radius=dev(rad), scale=1.1, visit_stride=stride)
        check_status(h)
        g = {k2: host(v) for k2, v in g.items()}
        o = oracle.search(wl.index, qs, nprobe, 50, radius=rad, scale=1.1, dumps=True, visit_stride=stride)
        assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
        assert_visits_parity(g, o, wl.index.nsub)
        assert_topk_parity(g["dist"], g["ids"], o["dist"], o["ids"])
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("base,kw", [("c3", {}), ("c4", {})])
def test_wide_shapes_two_clusters_per_build_pass(base, kw, monkeypatch):
    """48 x 2 and 50 x 4 have a second kernel arrangement (the tables of two probed clusters built in
    one pass over the codebook), chosen when the index is loaded: top-k parity for odd and even probe
    counts, splits, both count scores, and the stage dumps."""
    monkeypatch.setenv("IVFPQ_ROT_KERNEL", "pair")
    wl = Workload(small_cfg(base, n=30_000, ncomp=300, nlist=96, nq=60, chunk=16384, kmeans_iters=4, **kw))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nprobe, k, nsplit in ((7, 100, 1), (8, 1000, 1), (1, 10, 1), (9, 50, 2)):
            lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
            d, i = lib.ivfpq_search_dense(h, q, nprobe, k)
            o = oracle.search(wl.index, wl.queries, nprobe, k, dense=True)
            check_status(h)
            assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
            for score in (0, 1, 2):
                d, i = lib.ivfpq_search_sparse(h, q, nprobe, dev(wl.radius_per_query), k, scale=0.9, score=score)
                o = oracle.search(wl.index, wl.queries, nprobe, k, radius=wl.radius_per_query, scale=0.9, score=score)
                check_status(h)
                assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 0)
        nq, nprobe, stride = 16, 5, 8000
        qs, rad = wl.queries[:nq], wl.radius_per_query[:nq]
        g = lib.ivfpq_debug_search(h, dev(qs), nprobe, 50, radius=dev(rad), scale=1.1, visit_stride=stride)
        check_status(h)
        g = {k2: host(v) for k2, v in g.items()}
        o = oracle.search(wl.index, qs, nprobe, 50, radius=rad, scale=1.1, dumps=True, visit_stride=stride)
        assert np.array_equal(g["masks"].view(np.uint32), o["masks"])
        assert_visits_parity(g, o, wl.index.nsub)
        assert_topk_parity(g["dist"], g["ids"], o["dist"], o["ids"])
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("kernel", ["warps16", "warps32"])
def test_16x8_many_probes_and_splits(kernel, monkeypatch):
    """More probed clusters than the kernels stage at a time (128), alone and split over several
    CTAs per query, on an index with short and empty lists."""
    monkeypatch.setenv("IVFPQ_SCAN_KERNEL", kernel)
    wl = Workload(small_cfg("c1", n=20_000, ncomp=200, nlist=300, nq=24, chunk=16384, kmeans_iters=3))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        for nsplit in (1, 3):
            lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
            for nprobe, k in ((200, 100), (300, 1000), (129, 7)):
                d, i = lib.ivfpq_search_sparse(h, q, nprobe, dev(wl.radius), k, scale=1.0)
                check_status(h)
                o = oracle.search(wl.index, wl.queries, nprobe, k, radius=wl.radius, scale=1.0)
                assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 0)
        d, i = lib.ivfpq_search_dense(h, q, 256, 1024)
        check_status(h)
        o = oracle.search(wl.index, wl.queries, 256, 1024, dense=True)
        assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("mode", ["per_subspace", "per_query"])
@pytest.mark.parametrize("scale,penalty", [(1.0, -1.0), (0.5, -1.0), (2.0, 123.5), (0.0, 3.0), (float("inf"), -1.0)])
def test_sparse_search_matches_oracle(loaded, mode, scale, penalty):
    wl, h = loaded["small"]
    rad = wl.radius if mode == "per_subspace" else wl.radius_per_query
    d, i = lib.ivfpq_search_sparse(h, dev(wl.queries), 6, dev(rad), 40, scale=scale, miss_penalty=penalty)
    check_status(h)
    o = oracle.search(wl.index, wl.queries, 6, 40, radius=rad, scale=scale, miss_penalty=penalty)
    assert_topk_parity(host(d), host(i), o["dist"], o["ids"])


def test_infinite_radius_equals_dense_on_gpu(loaded):
    wl, h = loaded["pq2"]
    q = dev(wl.queries)
    d0, i0 = lib.ivfpq_search_dense(h, q, 5, 30)
    d1, i1 = lib.ivfpq_search_sparse(h, q, 5, dev(np.full(wl.index.nsub, np.inf, F32)), 30)
    assert torch.equal(i0, i1) and torch.equal(d0.view(torch.int32), d1.view(torch.int32))


def test_mixed_infinite_radius_reports_inf_with_valid_ids(loaded):
    wl, h = loaded["small"]
    rad = wl.radius.copy() * 0.5
    rad[0] = np.inf
    q = wl.queries[:16]
    d, i = lib.ivfpq_search_sparse(h, dev(q), 4, dev(rad), 1000)
    o = oracle.search(wl.index, q, 4, 1000, radius=rad)
    gd, gi = host(d), host(i)
    finite = np.isfinite(o["dist"])
    assert np.array_equal(np.isfinite(gd), finite)
    assert (np.isinf(gd) & (gi >= 0)).any()
    for qi in range(len(q)):
        n = int(finite[qi].sum())
        assert_topk_parity(gd[qi:qi + 1, :n], gi[qi:qi + 1, :n], o["dist"][qi:qi + 1, :n], o["ids"][qi:qi + 1, :n])
        # among +inf distances the order is by ascending id on both sides
        assert np.array_equal(gi[qi, n:], o["ids"][qi, n:])


@pytest.mark.parametrize("nsplit", [1, 2, 3, 8])
def test_probe_split_does_not_change_results(loaded, nsplit):
    wl, h = loaded["small"]
    q = dev(wl.queries)
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 1)
    d0, i0 = lib.ivfpq_search_sparse(h, q, 8, dev(wl.radius), 100)
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, nsplit)
    d1, i1 = lib.ivfpq_search_sparse(h, q, 8, dev(wl.radius), 100)
    lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 0)
    check_status(h)
    assert torch.equal(i0, i1) and torch.equal(d0.view(torch.int32), d1.view(torch.int32))
    o = oracle.search(wl.index, wl.queries, 8, 100, radius=wl.radius)
    assert_topk_parity(host(d1), host(i1), o["dist"], o["ids"])


def test_hand_worked_example_on_gpu():
    idx = hand_index()
    h = lib.ivfpq_index_load(idx)
    q = dev(np.array([[1.0, 1.0]], F32))
    d, i = lib.ivfpq_search_dense(h, q, 2, 5)
    assert host(i).tolist() == [[3, 5, 7, 1, 9]] and host(d).tolist() == [[0.0, 5.0, 10.0, 100.0, 181.0]]
    d, i = lib.ivfpq_search_sparse(h, q, 2, dev(np.array([2.0, 1.0], F32)), 5)
    assert host(i).tolist() == [[3, 5, 7, 1, 9]] and host(d).tolist() == [[0.0, 6.0, 6.0, 10.0, 10.0]]
    d, i = lib.ivfpq_search_dense(h, q, 1, 4)
    assert host(i).tolist() == [[3, 5, 7, -1]] and np.isinf(host(d)[0, 3])
    lib.ivfpq_index_free(h)


def test_edge_cases_small_codebook_empty_lists_single_query():
    # ksub = 16 (< 256), several empty lists, k larger than anything visited
    idx, base = lossless_toy_index(seed=2, n=300, nlist=150, nsub=5, dsub=3, ksub=16, spread=3.0)
    assert (np.diff(idx.list_offsets) == 0).any()
    h = lib.ivfpq_index_load(idx)
    rng = np.random.default_rng(1)
    q = (base[rng.integers(0, 300, 9)] + rng.standard_normal((9, idx.d))).astype(F32)
    for nq in (1, 9):
        for nprobe, k in ((150, 400), (3, 7), (1, 1024)):
            d, i = lib.ivfpq_search_dense(h, dev(q[:nq]), nprobe, k)
            assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
            o = oracle.search(idx, q[:nq], nprobe, k, dense=True)
            assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
            rad = np.full(idx.nsub, 1.5, F32)
            d, i = lib.ivfpq_search_sparse(h, dev(q[:nq]), nprobe, dev(rad), k)
            o = oracle.search(idx, q[:nq], nprobe, k, radius=rad)
            assert_topk_parity(host(d), host(i), o["dist"], o["ids"])
    lib.ivfpq_index_free(h)


def test_host_buffer_entry_point_matches_device_entry_point(loaded):
    wl, h = loaded["small"]
    nq, k = wl.queries.shape[0], 25
    qh = torch.from_numpy(wl.queries).pin_memory()
    od = torch.empty((nq, k), dtype=torch.float32).pin_memory()
    oi = torch.empty((nq, k), dtype=torch.int32).pin_memory()
    lib.ivfpq_search_host(h, qh, 5, k, od, oi, radius=dev(wl.radius), scale=1.2)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    d, i = lib.ivfpq_search_sparse(h, dev(wl.queries), 5, dev(wl.radius), k, scale=1.2)
    torch.cuda.synchronize()
    assert np.array_equal(od.numpy(), host(d)) and np.array_equal(oi.numpy(), host(i))
    lib.ivfpq_search_host(h, qh, 5, k, od, oi)
    torch.cuda.synchronize()
    d, i = lib.ivfpq_search_dense(h, dev(wl.queries), 5, k)
    assert np.array_equal(od.numpy(), host(d)) and np.array_equal(oi.numpy(), host(i))


@pytest.mark.parametrize("nq", [2048, 5003])
def test_host_entry_point_in_slices(loaded, nq):
    """Large batches go through the host entry point in slices (transfers of one slice overlap
    the search of another): same results as one device call, per-query radii follow their slice,
    the status covers every slice."""
    wl, h = loaded["small"]
    rng = np.random.default_rng(nq)
    pick = rng.integers(0, wl.queries.shape[0], nq)
    q = np.ascontiguousarray(wl.queries[pick] + rng.standard_normal((nq, wl.queries.shape[1])).astype(F32) * 0.01)
    rad = np.ascontiguousarray(wl.radius_per_query[pick] * (1 + 0.1 * rng.random((nq, wl.index.nsub), dtype=F32)))
    k = 25
    qh = torch.from_numpy(q).pin_memory()
    od = torch.empty((nq, k), dtype=torch.float32).pin_memory()
    oi = torch.empty((nq, k), dtype=torch.int32).pin_memory()
    for radius in (None, dev(rad), dev(wl.radius)):
        od.fill_(-1.0)
        oi.fill_(-7)
        lib.ivfpq_search_host(h, qh, 5, k, od, oi, radius=radius, scale=0.9)
        check_status(h)   # synchronises the stream
        if radius is None:
            d, i = lib.ivfpq_search_dense(h, dev(q), 5, k)
        else:
            d, i = lib.ivfpq_search_sparse(h, dev(q), 5, radius, k, scale=0.9)
        check_status(h)
        assert np.array_equal(oi.numpy(), host(i))
        assert np.array_equal(od.numpy().view(np.uint32), host(d).view(np.uint32))
    # against the oracle on a sample, and a bad probe count still fails up front
    sel = np.sort(rng.choice(nq, 64, replace=False))
    o = oracle.search(wl.index, q[sel], 5, k, radius=wl.radius, scale=0.9)
    assert_topk_parity(od.numpy()[sel], oi.numpy()[sel], o["dist"], o["ids"])
    with pytest.raises(lib.IvfpqError):
        lib.ivfpq_search_host(h, qh, wl.index.nlist + 1, k, od, oi)


def test_error_codes_on_gpu(loaded):
    wl, h = loaded["small"]
    q = dev(wl.queries)
    L = lib.load_library()
    ws = torch.empty(lib.ivfpq_search_workspace_bytes(h, q.shape[0], 4, 10), dtype=torch.uint8, device="cuda")
    od = torch.empty((q.shape[0], 10), dtype=torch.float32, device="cuda")
    oi = torch.empty((q.shape[0], 10), dtype=torch.int32, device="cuda")
    args = lambda **kw: [h.handle, kw.get("q", q.data_ptr()), kw.get("nq", q.shape[0]), kw.get("nprobe", 4),
                         kw.get("k", 10), od.data_ptr(), oi.data_ptr(), kw.get("ws", ws.data_ptr()),
                         kw.get("wsb", ws.numel()), None]
    assert L.ivfpq_search_dense(*args()) == lib.IVFPQ_OK
    assert L.ivfpq_search_dense(*args(k=2000)) == lib.IVFPQ_ERR_UNSUPPORTED
    assert L.ivfpq_search_dense(*args(nprobe=wl.index.nlist + 1)) == lib.IVFPQ_ERR_UNSUPPORTED
    assert L.ivfpq_search_dense(*args(nq=0)) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_search_dense(*args(q=None)) == lib.IVFPQ_ERR_INVALID_ARGUMENT
    assert L.ivfpq_search_dense(*args(wsb=128)) == lib.IVFPQ_ERR_WORKSPACE
    assert L.ivfpq_search_dense(*args(ws=ws.data_ptr() + 4)) == lib.IVFPQ_ERR_WORKSPACE
    torch.cuda.synchronize()
    with pytest.raises(lib.IvfpqError):
        lib.ivfpq_search_dense(h, q, 4, 5000)


def _full_size_parity(cfg_name, nprobe, nsample, scale):
    from ivfpq_inputs import CONFIGS
    wl = Workload(CONFIGS[cfg_name], device="cuda")
    h = lib.ivfpq_index_load(wl.index)
    q_all = dev(wl.queries)
    k = wl.cfg.k
    # the launch configuration the benchmark times: the whole query batch in one call
    d, i = lib.ivfpq_search_sparse(h, q_all, nprobe, dev(wl.radius), k, scale=scale)
    dd, di = lib.ivfpq_search_dense(h, q_all, nprobe, k)
    assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
    rng = np.random.default_rng(0)
    sel = np.sort(rng.choice(wl.queries.shape[0], nsample, replace=False))
    o = oracle.search(wl.index, wl.queries[sel], nprobe, k, radius=wl.radius, scale=scale)
    assert_topk_parity(host(d)[sel], host(i)[sel], o["dist"], o["ids"])
    o = oracle.search(wl.index, wl.queries[sel], nprobe, k, dense=True)
    assert_topk_parity(host(dd)[sel], host(di)[sel], o["dist"], o["ids"])
    if (wl.index.nsub, wl.index.dsub) == (16, 8):
        # the walk through the entry -> points map at full size (lists of several 8192-point chunks on the
        # 100 M-point workload): same answers as the code stream on a slice of the batch
        n = 256
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, lib.IVFPQ_SPARSE_SCAN_MAP)
        md, mi = lib.ivfpq_search_sparse(h, q_all[:n].contiguous(), nprobe, dev(wl.radius), k, scale=scale)
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_SPARSE_SCAN, lib.IVFPQ_SPARSE_SCAN_AUTO)
        assert lib.ivfpq_sync_status(h) == lib.IVFPQ_OK
        assert_topk_parity(host(md), host(mi), host(d)[:n], host(i)[:n])
    # properties that hold at any size: ascending, no duplicate ids, ids in range
    gi = host(di)
    assert (np.diff(host(dd), axis=1) >= 0).all()
    assert gi.min() >= 0 and gi.max() < wl.index.ntotal
    srt = np.sort(gi, axis=1)
    assert (np.diff(srt, axis=1) > 0).all()
    lib.ivfpq_index_free(h)


def test_full_size_c1_all_queries():
    _full_size_parity("c1", 8, 1000, 1.0)


def test_full_size_c3_sampled_queries():
    _full_size_parity("c3", 16, 64, 1.0)


def test_full_size_c4_sampled_queries():
    _full_size_parity("c4", 32, 48, 1.0)


def test_full_size_c5_sampled_queries():
    """100 M points (1.6 GB of codes, built in streamed chunks on the GPU): the whole 10 k-query
    batch in one call as the benchmark does, a sample of it checked against the oracle."""
    _full_size_parity("c5", 32, 24, 1.0)


def test_full_size_c2_sampled_queries():
    _full_size_parity("c2", 16, 128, 1.0)


@pytest.mark.parametrize("name", ["16x8", "48x2", "50x4", "10x3"])
def test_production_instances_equal_stage_dump_instances(shaped, name):
    """The stage dumps come from kernel instances of their own (compiled with the dump code, score read
    at run time, no early abandon); the instances that serve the search calls must return the same
    top-k bit for bit, for the dense search and for every score of the sparse one."""
    wl, h = shaped[name]
    q = dev(wl.queries)
    rad = dev(wl.radius_per_query)
    for nprobe, k in ((6, 100), (11, 17)):
        d, i = lib.ivfpq_search_dense(h, q, nprobe, k)
        g = lib.ivfpq_debug_search(h, q, nprobe, k)
        check_status(h)
        assert torch.equal(i, g["ids"]) and torch.equal(d.view(torch.int32), g["dist"].view(torch.int32))
        for score in (0, 1, 2):
            d, i = lib.ivfpq_search_sparse(h, q, nprobe, rad, k, scale=0.9, score=score)
            g = lib.ivfpq_debug_search(h, q, nprobe, k, radius=rad, scale=0.9, score=score)
            check_status(h)
            assert torch.equal(i, g["ids"]) and torch.equal(d.view(torch.int32), g["dist"].view(torch.int32))


@pytest.mark.parametrize("kernel", ["warps16", "warps32"])
def test_16x8_production_instances_equal_stage_dump_instances(kernel, monkeypatch):
    """Same as above for both persistent instances of the 16 x 8 shape; the 32-warp one abandons
    blocks early in its production form and never in its stage-dump form: same top-k bit for bit."""
    monkeypatch.setenv("IVFPQ_SCAN_KERNEL", kernel)
    wl = Workload(small_cfg("c1", n=40_000, ncomp=300, nlist=64, nq=70, chunk=16384, kmeans_iters=4))
    h = lib.ivfpq_index_load(wl.index)
    try:
        q = dev(wl.queries)
        lib.ivfpq_index_set_option(h, lib.IVFPQ_OPT_NSPLIT, 1)
        for nprobe, k in ((9, 100), (30, 10)):
            d, i = lib.ivfpq_search_dense(h, q, nprobe, k)
            g = lib.ivfpq_debug_search(h, q, nprobe, k)
            check_status(h)
            assert torch.equal(i, g["ids"]) and torch.equal(d.view(torch.int32), g["dist"].view(torch.int32))
            for score, scale in ((0, 0.6), (0, 1.0), (1, 0.8), (2, 1.2)):
                d, i = lib.ivfpq_search_sparse(h, q, nprobe, dev(wl.radius), k, scale=scale, score=score)
                g = lib.ivfpq_debug_search(h, q, nprobe, k, radius=dev(wl.radius), scale=scale, score=score)
                check_status(h)
                assert torch.equal(i, g["ids"]) and torch.equal(d.view(torch.int32), g["dist"].view(torch.int32))
    finally:
        lib.ivfpq_index_free(h)
