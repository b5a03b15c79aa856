"""Comparison rules between the CUDA path and the CPU oracle.

Integer decisions (probe lists, selected-entry masks, per-point hit sets) must be
bit-equal.  fp32 distances must agree within RTOL relative (the two sides may sum
the subspace terms in different orders).  Top-k id lists must be identical except
for candidates whose distances are within RTOL of each other or of the k-th
distance, where either order (or either member across the cut) is acceptable.
"""

import numpy as np

RTOL = 1e-4


def close(a, b, rtol=RTOL, floor=0.0):
    """|a - b| <= rtol * max(|a|, |b|, floor).  `floor` (a magnitude) is for sums of terms of both
    signs (inner products), whose rounding error scales with the terms, not with the result."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    both_inf = np.isinf(a) & np.isinf(b) & (np.sign(a) == np.sign(b))
    with np.errstate(invalid="ignore"):
        ok = np.abs(a - b) <= rtol * np.maximum(np.maximum(np.abs(a), np.abs(b)), floor)
    return ok | both_inf


def assert_topk_parity(g_dist, g_ids, o_dist, o_ids, rtol=RTOL, floor=0.0):
    """g_*: CUDA results, o_*: oracle results, [nq, k]."""
    g_dist, g_ids, o_dist, o_ids = map(np.asarray, (g_dist, g_ids, o_dist, o_ids))
    assert g_dist.shape == o_dist.shape and g_ids.shape == o_ids.shape
    bad = ~close(g_dist, o_dist, rtol, floor)
    assert not bad.any(), f"distance mismatch at {np.argwhere(bad)[:5]}: {g_dist[bad][:5]} vs {o_dist[bad][:5]}"
    # ascending, ties by ascending id, padding at the end
    finite = np.nan_to_num(g_dist, posinf=float(np.finfo(np.float32).max))
    assert (np.diff(finite, axis=1) >= 0).all(), "distances must ascend"
    same_d = (g_dist[:, 1:] == g_dist[:, :-1]) & (g_ids[:, 1:] >= 0) & (g_ids[:, :-1] >= 0)
    assert (g_ids[:, 1:][same_d] > g_ids[:, :-1][same_d]).all(), "equal distances must be ordered by id"
    assert ((g_ids == -1) == (o_ids == -1)).all(), "padding differs"
    assert (np.isinf(g_dist[g_ids == -1])).all()
    exact = (g_ids == o_ids).all(axis=1)
    for qi in np.nonzero(~exact)[0]:
        gd, gi, od, oi = g_dist[qi], g_ids[qi], o_dist[qi], o_ids[qi]
        gmap = dict(zip(gi.tolist(), gd.tolist()))
        omap = dict(zip(oi.tolist(), od.tolist()))
        valid = oi >= 0
        kth = float(od[valid][-1]) if valid.any() else np.inf
        for i, d in omap.items():
            if i < 0:
                continue
            if i in gmap:
                assert close(gmap[i], d, rtol, floor), (qi, i, gmap[i], d)
            else:       # dropped across the cut: must be within tolerance of the k-th distance
                assert close(d, kth, 2 * rtol, floor), (qi, i, d, kth)
        for i, d in gmap.items():
            if i >= 0 and i not in omap:
                assert close(d, kth, 2 * rtol, floor), (qi, i, d, kth)
        # position changes only among near-equal distances
        for pos in np.nonzero(gi != oi)[0]:
            assert close(gd[pos], od[pos], rtol, floor), (qi, pos)


def assert_visits_parity(g, o, nsub, rtol=RTOL, floor=0.0):
    """Per-visited-point dumps: ids and hit sets bit-equal, distances within rtol."""
    gc, oc = np.asarray(g["visit_count"]), np.asarray(o["visit_count"])
    assert np.array_equal(gc, oc)
    stride = o["visit_ids"].shape[1]
    for qi in range(len(oc)):
        n = min(int(oc[qi]), stride)
        assert np.array_equal(np.asarray(g["visit_ids"])[qi, :n], o["visit_ids"][qi, :n])
        gh = np.asarray(g["visit_hits"])[qi, :n].astype(np.uint64)
        assert np.array_equal(gh, o["visit_hits"][qi, :n]), f"hit sets differ for query {qi}"
        gd, od = np.asarray(g["visit_dist"])[qi, :n], o["visit_dist"][qi, :n]
        bad = ~close(gd, od, rtol, floor)
        assert not bad.any(), (qi, gd[bad][:4], od[bad][:4])
