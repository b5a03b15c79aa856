"""Pins for the entry usage / locality statistics of the CPU oracle (paper Sec. 3.2 and 3.3: which
codebook entries the neighbours of a query use, and how close those entries are to the query's
projection): a hand-worked example, counting invariants, the tie rule, a lossless index, and an
integer-valued case checked against numpy's sort."""

import numpy as np
import pytest

import oracle
from ivfpq_inputs import IvfPqIndex, lossless_toy_index
from test_oracle_pins import _golden, hand_index

F32 = np.float32


def test_hand_worked_usage_and_ranks():
    g = _golden("entry_stats_example.txt")
    ints = lambda k: [int(x) for x in g[k].split()]
    idx = hand_index()
    q = np.array([[1.0, 1.0]], F32)
    usage, hist = oracle.entry_stats(idx, q, np.array([ints("neighbors")], np.int64))
    assert usage[0].tolist() == ints("usage")
    assert hist[0].tolist() == ints("rank_hist0") and hist[1].tolist() == ints("rank_hist1")
    pos = np.array([ints("neighbors")[:3] + [-1]], np.int64)
    usage, hist = oracle.entry_stats(idx, q, pos)
    assert usage[0].tolist() == ints("usage3")
    assert hist[0].tolist() == ints("rank3_hist0") and hist[1].tolist() == ints("rank3_hist1")


def test_counting_invariants(wl_small):
    idx, q = wl_small.index, wl_small.queries[:40]
    rng = np.random.default_rng(0)
    pos = rng.integers(0, idx.ntotal, (40, 25)).astype(np.int64)
    pos[::3, 20:] = -1
    pos[5] = -1
    pos[7] = pos[7, 0]                                   # the same neighbour 25 times
    usage, hist = oracle.entry_stats(idx, q, pos)
    nvalid = (pos >= 0).sum(axis=1)
    assert (hist.sum(axis=1) == nvalid.sum()).all()      # one count per (query, neighbour) and subspace
    assert (usage <= np.minimum(nvalid, idx.ksub)[:, None]).all()
    assert (usage[nvalid > 0] >= 1).all() and (usage[5] == 0).all() and (usage[7] == 1).all()
    # distinct codes of the neighbours, straight from the code array
    for i in (0, 1, 2, 11):
        v = pos[i][pos[i] >= 0]
        assert usage[i].tolist() == [len(set(idx.codes[v, s].tolist())) for s in range(idx.nsub)]


def test_ties_are_ordered_by_entry_number():
    """Two identical entries: the one with the smaller number counts as closer."""
    cent = np.zeros((1, 1), F32)
    cb = np.array([[[5.0], [2.0], [2.0], [9.0]]], F32)
    codes = np.array([[1], [2]], np.uint8)
    idx = IvfPqIndex(d=1, nlist=1, nsub=1, dsub=1, ksub=4, ntotal=2, coarse_centroids=cent, codebooks=cb,
                     list_offsets=np.array([0, 2], np.int64), codes=codes, ids=np.array([0, 1], np.int32))
    q = np.array([[2.0]], F32)
    _, hist = oracle.entry_stats(idx, q, np.array([[0]], np.int64))
    assert hist[0].tolist() == [1, 0, 0, 0]              # entry 1: nothing before it
    _, hist = oracle.entry_stats(idx, q, np.array([[1]], np.int64))
    assert hist[0].tolist() == [0, 1, 0, 0]              # entry 2: its twin, entry 1, comes first
    # at q = 7 entries 0 and 3 are equally far (4): entry 0 first
    codes[0, 0], codes[1, 0] = 0, 3
    _, hist = oracle.entry_stats(idx, np.array([[7.0]], F32), np.array([[0, 1]], np.int64))
    assert hist[0].tolist() == [1, 1, 0, 0]


def test_a_base_point_of_a_lossless_index_uses_its_closest_entries():
    idx, base = lossless_toy_index(seed=9, n=300, nlist=6, nsub=3, dsub=2, ksub=32, spread=6.0)
    pos_of_id = np.empty(idx.ntotal, np.int64)
    pos_of_id[idx.ids] = np.arange(idx.ntotal)
    pick = np.arange(0, 300, 7)
    usage, hist = oracle.entry_stats(idx, base[pick], pos_of_id[pick][:, None])
    assert (usage == 1).all()
    assert (hist[:, 0] == len(pick)).all() and hist[:, 1:].sum() == 0


def test_integer_case_against_numpy_sort():
    """Small-integer coordinates make every distance exact in fp32 and fp64 alike: the rank must be
    the position of the entry in numpy's stable sort of the fp64 distances."""
    rng = np.random.default_rng(4)
    nlist, nsub, dsub, ksub, n, nq, k = 5, 4, 3, 64, 200, 30, 12
    d = nsub * dsub
    cent = rng.integers(-20, 20, (nlist, d)).astype(F32)
    cb = rng.integers(-8, 8, (nsub, ksub, dsub)).astype(F32)
    sizes = rng.multinomial(n, np.ones(nlist) / nlist)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    codes = rng.integers(0, ksub, (n, nsub)).astype(np.uint8)
    idx = IvfPqIndex(d=d, nlist=nlist, nsub=nsub, dsub=dsub, ksub=ksub, ntotal=n, coarse_centroids=cent,
                     codebooks=cb, list_offsets=off, codes=codes, ids=np.arange(n, dtype=np.int32))
    q = rng.integers(-25, 25, (nq, d)).astype(F32)
    pos = rng.integers(0, n, (nq, k)).astype(np.int64)
    usage, hist = oracle.entry_stats(idx, q, pos)
    want = np.zeros((nsub, ksub), np.int64)
    for i in range(nq):
        for x in pos[i]:
            c = int(np.searchsorted(off, x, side="right") - 1)
            for s in range(nsub):
                res = q[i, s * dsub:(s + 1) * dsub].astype(np.float64) - cent[c, s * dsub:(s + 1) * dsub]
                dist = ((res[None, :] - cb[s].astype(np.float64)) ** 2).sum(axis=1)
                order = np.argsort(dist, kind="stable")
                want[s, int(np.nonzero(order == codes[x, s])[0][0])] += 1
    assert np.array_equal(hist, want)
    assert len(np.unique(np.nonzero(hist)[1])) > 20


def test_exact_neighbours_use_few_and_close_entries(wl_small):
    """The two observations of Sec. 3.2 / 3.3 on the synthetic mixture: the exact neighbours of a
    query use a minority of the entries, and those entries are among the closest ones."""
    from ivfpq_inputs import CONFIGS  # noqa: F401  (same recipe as the benchmark configs)
    idx, q = wl_small.index, wl_small.queries[:32]
    # neighbours under the quantized metric stand in for the exact ones (no raw vectors kept here)
    o = oracle.search(idx, q, idx.nlist, 50, dense=True)
    pos_of_id = np.empty(idx.ntotal, np.int64)
    pos_of_id[idx.ids] = np.arange(idx.ntotal)
    usage, hist = oracle.entry_stats(idx, q, pos_of_id[o["ids"]])
    assert usage.mean() / idx.ksub < 0.3
    cdf = np.cumsum(hist.sum(axis=0)) / hist.sum()
    assert cdf[idx.ksub // 2 - 1] > 0.9
