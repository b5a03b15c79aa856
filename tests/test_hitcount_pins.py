"""Pins for the hit-count scores of the CPU oracle (paper Sec. 5.4 "Aggressive Approximation: hit
count-based Method"): values worked by hand, limits in which the score is known in closed form, and
identities that tie the counts to the distance mode, which has pins of its own."""

import numpy as np
import pytest

import oracle
from test_oracle_pins import _golden, hand_index

F32 = np.float32


def test_hand_worked_hit_count_and_reward_penalty():
    g = _golden("hand_example.txt")
    nums = lambda k: [float(x) for x in g[k].split()]
    idx = hand_index()
    q = np.array([nums("query")], F32)
    rad = np.array(nums("radius"), F32)
    o = oracle.search(idx, q, 2, 5, radius=rad, score=1)
    assert o["ids"][0].tolist() == nums("count_ids") and o["dist"][0].tolist() == nums("count_value")
    o = oracle.search(idx, q, 2, 5, radius=rad, score=2)
    assert o["ids"][0].tolist() == nums("reward_ids") and o["dist"][0].tolist() == nums("reward_value")


def _visited_ids(idx, probes):
    off = idx.list_offsets
    return np.concatenate([idx.ids[off[c]:off[c + 1]] for c in probes])


@pytest.mark.parametrize("score", [1, 2])
def test_limits_all_hit_and_all_missed(wl_small, score):
    """Radius -> infinity: every subspace is an (inner) hit, value 0 for every visited point, so
    the answer is the k smallest ids of the probed lists.  Radius 0 with no exact zero distance:
    every subspace missed, value nsub (hit count) or 2 nsub (reward/penalty), same ids."""
    idx, q = wl_small.index, wl_small.queries[:24]
    k, nprobe = 30, 4
    pid, _ = oracle.coarse(idx, q, nprobe)
    for radius, value in ((np.inf, 0.0), (0.0, float(idx.nsub * score))):
        o = oracle.search(idx, q, nprobe, k, radius=np.full(idx.nsub, radius, F32), score=score)
        for i in range(q.shape[0]):
            want = np.sort(_visited_ids(idx, pid[i]))[:k]
            assert o["ids"][i].tolist() == want.tolist()
            assert (o["dist"][i] == value).all()


def test_hit_count_equals_miss_count_of_the_distance_mode(wl_small):
    """Distance mode with a penalty P far above any sum of table values reports S + m P with
    S < P, so floor(dist / P) is the number m of missed subspaces of that point; the hit-count
    score must report the same m for the same point (every visited point, through the dumps)."""
    idx, q = wl_small.index, wl_small.queries[:32]
    P = 2.0 ** 40
    kw = dict(radius=wl_small.radius, scale=0.8, visit_stride=6000)
    h = oracle.search(idx, q, 5, 10, miss_penalty=P, **kw)
    c = oracle.search(idx, q, 5, 10, score=1, **kw)
    n = int(min(h["visit_count"].min(), 6000))
    assert n > 500
    assert np.array_equal(h["visit_ids"][:, :n], c["visit_ids"][:, :n])
    m = np.floor(h["visit_dist"][:, :n].astype(np.float64) / P)
    assert np.array_equal(m, c["visit_dist"][:, :n].astype(np.float64))
    # and the hit sets give the same count
    pop = np.array([[bin(int(x)).count("1") for x in row[:n]] for row in c["visit_hits"]])
    assert np.array_equal(idx.nsub - pop, m)
    assert 0 < m.mean() < idx.nsub


def test_reward_penalty_is_the_sum_of_two_miss_counts(wl_small):
    """0 / 1 / 2 per subspace (inner hit / outer only / missed) = [missed the outer sphere] +
    [missed the inner sphere]: the reward/penalty value at radius r equals the hit-count value at
    r plus the hit-count value at r / 2 (halving is exact in fp32), point by point."""
    idx, q = wl_small.index, wl_small.queries[:32]
    kw = dict(radius=wl_small.radius_per_query[:32], visit_stride=5000)
    outer = oracle.search(idx, q, 4, 10, score=1, scale=1.5, **kw)
    inner = oracle.search(idx, q, 4, 10, score=1, scale=0.75, **kw)
    both = oracle.search(idx, q, 4, 10, score=2, scale=1.5, **kw)
    n = int(min(both["visit_count"].min(), 5000))
    assert np.array_equal(both["visit_dist"][:, :n], outer["visit_dist"][:, :n] + inner["visit_dist"][:, :n])
    assert np.array_equal(both["visit_hits"], outer["visit_hits"])       # hit sets describe the outer sphere
    assert (inner["visit_dist"][:, :n] >= outer["visit_dist"][:, :n]).all()
    assert len(np.unique(both["visit_dist"][:, :n])) > 5


@pytest.mark.parametrize("score", [1, 2])
def test_top_k_is_the_sorted_prefix_of_all_visited_points(wl_pq2, score):
    idx, q = wl_pq2.index, wl_pq2.queries[:16]
    o = oracle.search(idx, q, 5, 40, radius=wl_pq2.radius, score=score, visit_stride=4000)
    for i in range(q.shape[0]):
        n = int(o["visit_count"][i])
        assert n <= 4000
        order = np.lexsort((o["visit_ids"][i, :n], o["visit_dist"][i, :n]))[:40]
        assert o["ids"][i].tolist() == o["visit_ids"][i, order].tolist()
        assert o["dist"][i].tolist() == o["visit_dist"][i, order].tolist()


def test_more_hits_means_closer_on_average(wl_small):
    """The observation the method rests on (Sec. 5.4): the hit count correlates with the distance.
    On the synthetic mixture the points ranked first by hit count are closer (dense ADC distance)
    than the visited points on average, and the reward/penalty score ranks at least as well."""
    idx, q = wl_small.index, wl_small.queries[:48]
    dense = oracle.search(idx, q, 6, 20, dense=True, visit_stride=6000)
    means = {}
    for score in (1, 2):
        o = oracle.search(idx, q, 6, 20, radius=wl_small.radius, score=score)
        got = []
        for i in range(q.shape[0]):
            n = int(min(dense["visit_count"][i], 6000))
            lut = dict(zip(dense["visit_ids"][i, :n].tolist(), dense["visit_dist"][i, :n].tolist()))
            got.append(np.mean([lut[j] for j in o["ids"][i].tolist() if j in lut]))
        means[score] = float(np.mean(got))
    allmean = float(np.mean([dense["visit_dist"][i, :int(min(dense["visit_count"][i], 6000))].mean() for i in range(48)]))
    assert means[1] < 0.6 * allmean and means[2] < 0.6 * allmean


def test_count_scores_need_a_radius(wl_small):
    with pytest.raises(ValueError):
        oracle.search(wl_small.index, wl_small.queries[:2], 2, 5, dense=True, score=1)
