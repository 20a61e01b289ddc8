"""Pins of the oracle's clustering steps (Fig. 4 steps 3, 4, 6)."""
import itertools

import numpy as np
import pytest


def brute_force_kmeans1d(v, w, k):
    n = len(v)
    best = np.inf
    for cuts in itertools.combinations(range(1, n), k - 1):
        b = (0,) + cuts + (n,)
        c = 0.0
        for i in range(k):
            vv, ww = v[b[i]:b[i + 1]], w[b[i]:b[i + 1]]
            mu = (vv * ww).sum() / ww.sum()
            c += (ww * (vv - mu) ** 2).sum()
        best = min(best, c)
    return best


@pytest.mark.parametrize("n,k", [(5, 2), (7, 3), (9, 3), (10, 2), (10, 3), (8, 4)])
def test_kmeans1d_dp_is_the_global_optimum(eo, n, k):
    rng = np.random.Generator(np.random.PCG64(n * 31 + k))
    for trial in range(5):
        v = np.sort(rng.standard_normal(n))
        if trial == 3:
            v[2] = v[1]                                 # duplicate values
        w = np.ones(n) if trial % 2 == 0 else rng.uniform(0.1, 3.0, n)
        cen, cost = eo.kmeans1d(v, k, None if trial % 2 == 0 else w)
        assert abs(cost - brute_force_kmeans1d(v, w, k)) < 1e-10
        assert np.all(np.diff(cen) >= 0)
        # the reported centroids realise the reported cost
        d = (v[:, None] - cen[None, :]) ** 2
        assert (w * d.min(axis=1)).sum() <= cost + 1e-10


def test_kmeans1d_beats_lloyd_and_matches_closed_forms(eo):
    rng = np.random.Generator(np.random.PCG64(3))
    v = np.sort(rng.standard_t(5, 127) * 0.2)
    cen, cost = eo.kmeans1d(v, 15)
    # k = n: zero cost, centroids are the points; k = 1: the variance
    c_all, cost_all = eo.kmeans1d(v, 127)
    assert cost_all < 1e-12 and np.allclose(c_all, v)
    c1, cost1 = eo.kmeans1d(v, 1)
    assert abs(c1[0] - v.mean()) < 1e-12 and abs(cost1 - ((v - v.mean()) ** 2).sum()) < 1e-9
    # any Lloyd run from quantile seeds is no better than the DP optimum
    c = np.quantile(v, (np.arange(15) + 0.5) / 15)
    for _ in range(50):
        a = np.abs(v[:, None] - c[None, :]).argmin(1)
        c = np.array([v[a == j].mean() if (a == j).any() else c[j] for j in range(15)])
    lloyd_cost = ((v - c[np.abs(v[:, None] - c[None, :]).argmin(1)]) ** 2).sum()
    assert cost <= lloyd_cost + 1e-12


def test_group_pattern_excludes_absmax_and_normalises_by_rounded_scale(eo):
    rng = np.random.Generator(np.random.PCG64(4))
    x = (rng.standard_normal(128) * 0.02).astype(np.float16)
    x[17] = np.float16(-0.3)                            # the abs-max, negative
    e = -10
    pat = eo.group_pattern(x, e)
    assert np.all(np.diff(pat) >= 0)
    s = abs(eo.e4m3_to_f32(eo.e4m3_from_f32(float(x[17]) / 2.0 ** e))) * 2.0 ** e
    u = np.sort(np.delete(x.astype(np.float32), 17) / np.float32(s)).astype(np.float64)
    cen, _ = eo.kmeans1d(u, 15)
    assert np.allclose(pat, cen)
    assert pat.min() >= u.min() and pat.max() <= u.max() and abs(pat).max() < 1.01


def test_lloyd_objective_never_increases_and_is_deterministic(eo):
    rng = np.random.Generator(np.random.PCG64(5))
    x = np.sort(rng.standard_normal((600, 15)), axis=1)
    cen, assign, trace, it = eo.lloyd(x, 8, seed=11, max_iter=25)
    t = trace[trace >= 0]
    assert len(t) >= 2 and np.all(np.diff(t) <= 1e-9)
    cen2, assign2, trace2, it2 = eo.lloyd(x, 8, seed=11, max_iter=25)
    assert np.array_equal(cen, cen2) and np.array_equal(assign, assign2)
    # means of ascending vectors are ascending: shared patterns stay sorted
    assert np.all(np.diff(cen, axis=1) >= 0)
    # the final assignment is the nearest centre, ties to the lower index
    d = ((x[:, None, :] - cen[None, :, :]) ** 2).sum(-1)
    if it < 25:
        assert np.array_equal(assign, d.argmin(1))
    # more clusters than distinct points: empty clusters are re-seeded, no crash, zero objective
    y = np.repeat(rng.standard_normal((3, 4)), 5, axis=0)
    cen3, a3, tr3, _ = eo.lloyd(y, 4, seed=2, max_iter=10)
    assert tr3[tr3 >= 0][-1] < 1e-12
