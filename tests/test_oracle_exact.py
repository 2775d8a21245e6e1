"""Pins of the oracle's exact 1-D weighted K-means (the optimum of the clustering objective, by dynamic
programming over the sorted row): brute force over all contiguous partitions of small rows, an independent numpy
DP, the two-cluster split scan, never worse than Lloyd, and the structure of its centroids."""
import itertools

import numpy as np
import pytest

from test_oracle_kmeans import _brute_two_clusters, _exact_kmeans_dp, _row


def _brute_partitions(x, g, k):
    order = np.argsort(x, kind="stable")
    xs, gs = x[order], g[order]
    m = len(xs)
    best = np.inf
    for cuts in itertools.combinations(range(1, m), k - 1):
        edges = (0,) + cuts + (m,)
        cost = 0.0
        for a, b in zip(edges[:-1], edges[1:]):
            w = gs[a:b].sum()
            if w > 0:
                mu = (gs[a:b] * xs[a:b]).sum() / w
                cost += (gs[a:b] * (xs[a:b] - mu) ** 2).sum()
        best = min(best, cost)
    return best


@pytest.mark.parametrize("seed", range(5))
def test_equals_brute_force_over_all_contiguous_partitions(oracle, seed):
    x, g = _row(300 + seed, 12, outliers=0.1)
    c, err = oracle.kmeans_exact_row(x, g, [2, 4, 8])
    scale = np.sum(g * x * x)
    for u, k in enumerate((2, 4, 8)):
        assert err[u] == pytest.approx(_brute_partitions(x, g, k), rel=1e-9, abs=1e-13 * scale)
    assert err[0] == pytest.approx(_brute_two_clusters(x, g), rel=1e-9)


@pytest.mark.parametrize("seed,m", [(1, 40), (2, 97), (3, 150)])
def test_equals_numpy_dp_and_never_worse_than_lloyd(oracle, seed, m):
    x, g = _row(400 + seed, m, outliers=0.05)
    ks = [2, 4, 8, 16]
    c, err = oracle.kmeans_exact_row(x, g, ks)
    scale = np.sum(g * x * x)
    off = 0
    for u, k in enumerate(ks):
        assert err[u] == pytest.approx(_exact_kmeans_dp(x, g, k), rel=1e-9, abs=1e-13 * scale)
        lloyd = oracle.kmeans_row(x, g, k, 60, round_fp32=False)
        assert err[u] <= lloyd["err"] + 1e-12 * scale
        ck = c[off:off + k]
        assert np.all(np.diff(ck) >= 0)
        # the centroids realise the optimum: nearest-centroid assignment costs what the DP says
        lab = np.argmin(np.abs(x[:, None] - ck[None, :]), axis=1)
        assert np.sum(g * (x - ck[lab]) ** 2) == pytest.approx(err[u], rel=1e-9, abs=1e-13 * scale)
        off += k
    assert np.all(np.diff(err) <= 1e-15 * scale)       # more clusters never cost more


def test_few_distinct_values_and_zero_weight(oracle):
    x = np.array([0.5, -1.0, 0.5, 2.0, -1.0, 0.5, -0.0, 0.0])
    g = np.arange(1.0, 9.0)
    c, err = oracle.kmeans_exact_row(x, g, [2, 4, 8])
    np.testing.assert_array_equal(c[2:6], [-1.0, 0.0, 0.5, 2.0])      # four distinct values (-0 and +0 are one)
    np.testing.assert_array_equal(c[6:14], [-1.0, 0.0, 0.5, 2.0, 2.0, 2.0, 2.0, 2.0])
    assert err[1] == 0.0 and err[2] == 0.0 and err[0] > 0.0
    # a stretch without weight costs nothing wherever it is cut; the weighted part decides
    x2 = np.array([0.0, 1.0, 2.0, 3.0, 10.0, 11.0])
    g2 = np.array([1.0, 1.0, 0.0, 0.0, 1.0, 1.0])
    c2, e2 = oracle.kmeans_exact_row(x2, g2, [2])
    assert e2[0] == pytest.approx(0.5 + 0.5)
    assert c2[1] == pytest.approx(10.5)


def test_matrix_wrapper_uses_the_clustered_values(oracle):
    from paper_2412_04180_b200 import inputs
    w, g = inputs.make_rows(6, 64, 3)
    s = inputs.make_scale(64, 4)
    res = oracle.cluster_rows_exact(w, g, [1, 2, 3], s=s)
    x = (w.astype(np.float32) * (np.float32(1.0) / s)).astype(np.float64)
    for i in range(6):
        c, err = oracle.kmeans_exact_row(x[i], g[i].astype(np.float64), [2, 4, 8])
        np.testing.assert_array_equal(res["centroids"][i], c)
        np.testing.assert_array_equal(res["err"][i], err)
    lloyd = oracle.cluster_rows(w, g, [1, 2, 3], 50, s=s, want_codes=False)
    assert np.all(res["err"] <= lloyd["err"] * (1 + 1e-12))
