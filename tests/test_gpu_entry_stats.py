"""GPU parity of the entry usage / locality statistics (paper Sec. 3.2, 3.3) against the CPU oracle:
both outputs are integer counts decided by fp32 distances taken in the same arithmetic, so the
comparison is exact."""

import numpy as np
import pytest
import torch

import oracle
import paper_2312_01712_b200 as lib
from conftest import Workload, small_cfg
from test_oracle_pins import _golden, hand_index

pytestmark = pytest.mark.gpu

F32 = np.float32


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_gpu(h, index, queries, pos):
    usage, hist, flags = lib.ivfpq_entry_stats(h, dev(index.codes), dev(queries), dev(pos))
    return usage.cpu().numpy(), hist.cpu().numpy(), flags


def test_hand_worked_statistics_on_gpu():
    g = _golden("entry_stats_example.txt")
    ints = lambda k: [int(x) for x in g[k].split()]
    idx = hand_index()
    h = lib.ivfpq_index_load(idx)
    try:
        usage, hist, flags = run_gpu(h, idx, np.array([[1.0, 1.0]], F32), np.array([ints("neighbors")], np.int64))
        assert flags == 0 and usage[0].tolist() == ints("usage")
        assert hist[0].tolist() == ints("rank_hist0") and hist[1].tolist() == ints("rank_hist1")
    finally:
        lib.ivfpq_index_free(h)


@pytest.mark.parametrize("name,base,kw", [
    ("16x8", "c1", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
    ("48x2", "c3", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
    ("50x4", "c4", dict(n=30_000, ncomp=300, nlist=96, nq=80)),
    ("10x3", "c4", dict(n=9_000, d=30, nsub=10, dsub=3, ncomp=100, nlist=37, nq=50)),
])
def test_statistics_identical_to_oracle(name, base, kw):
    wl = Workload(small_cfg(base, chunk=16384, kmeans_iters=4, **kw))
    idx, q = wl.index, wl.queries
    h = lib.ivfpq_index_load(idx)
    try:
        # neighbours under the quantized metric (all lists probed), plus random points and holes
        o = oracle.search(idx, q, idx.nlist, 100, dense=True)
        pos_of_id = np.empty(idx.ntotal, np.int64)
        pos_of_id[idx.ids] = np.arange(idx.ntotal)
        pos = pos_of_id[o["ids"]]
        rng = np.random.default_rng(1)
        pos[:, 90:] = rng.integers(0, idx.ntotal, (q.shape[0], 10))
        pos[::4, 70:80] = -1
        pos[3] = -1
        usage, hist, flags = run_gpu(h, idx, q, pos)
        ou, oh = oracle.entry_stats(idx, q, pos)
        assert flags == 0
        assert np.array_equal(usage, ou) and np.array_equal(hist, oh)
        assert hist.sum() == (pos >= 0).sum() * idx.nsub
        # accumulation into a histogram that already holds counts; a single neighbour per query
        again = torch.from_numpy(oh).cuda()
        _, hist2, _ = lib.ivfpq_entry_stats(h, dev(idx.codes), dev(q), dev(pos[:, :1]), rank_hist=again)
        ou1, oh1 = oracle.entry_stats(idx, q, pos[:, :1])
        assert np.array_equal(hist2.cpu().numpy(), oh + oh1)
    finally:
        lib.ivfpq_index_free(h)


def test_out_of_range_positions_are_flagged_and_skipped(wl_small):
    idx, q = wl_small.index, wl_small.queries[:10]
    h = lib.ivfpq_index_load(idx)
    try:
        rng = np.random.default_rng(2)
        pos = rng.integers(0, idx.ntotal, (10, 8)).astype(np.int64)
        bad = pos.copy()
        bad[2, 3] = idx.ntotal
        bad[7, 0] = idx.ntotal + 12345
        usage, hist, flags = run_gpu(h, idx, q, bad)
        assert flags != 0
        pos[2, 3] = pos[7, 0] = -1
        ou, oh = oracle.entry_stats(idx, q, pos)
        assert np.array_equal(usage, ou) and np.array_equal(hist, oh)
        with pytest.raises(lib.IvfpqError) as e:
            lib.ivfpq_entry_stats(h, dev(idx.codes), dev(q), dev(np.zeros((10, 2000), np.int64)))
        assert e.value.code == lib.IVFPQ_ERR_UNSUPPORTED
    finally:
        lib.ivfpq_index_free(h)
