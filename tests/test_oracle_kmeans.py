"""Pins for the CPU oracle's weighted 1-D K-means (no GPU, no CUDA code involved).

Each test checks the oracle against something fixed by the method's definition or by
mathematics: hand-worked examples, the monotone objective, the exact optimum from a
dynamic programme / brute force, a library K-means given the same init, exact symmetries.
"""
import itertools
import os

import numpy as np
import pytest

from paper_2412_04180_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "kmeans_hand_examples.txt")


def _hand_examples():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, xs, gs, k, iters, cs, err, labels = [p.strip() for p in line.split("|")]
            out.append((name, np.array(xs.split(), float), np.array(gs.split(), float), int(k), int(iters),
                        np.array(cs.split(), float), float(err), np.array(labels.split(), int)))
    return out


@pytest.mark.parametrize("ex", _hand_examples(), ids=lambda e: e[0])
@pytest.mark.parametrize("round_fp32", [True, False])
def test_hand_worked_examples(oracle, ex, round_fp32):
    _, x, g, k, iters, c, err, labels = ex
    r = oracle.kmeans_row(x, g, k, iters, round_fp32=round_fp32)
    np.testing.assert_allclose(r["c"], c, rtol=0, atol=1e-12)
    assert r["err"] == pytest.approx(err, abs=1e-9)
    np.testing.assert_array_equal(r["label"], labels)


def _row(seed, m, sigma_g=1.5, outliers=1e-3):
    w, g = inputs.make_rows(1, m, seed, importance_sigma=sigma_g, outlier_frac=outliers)
    return w[0].astype(np.float64), g[0].astype(np.float64)


@pytest.mark.parametrize("round_fp32", [True, False])
@pytest.mark.parametrize("seed,m", [(1, 512), (2, 4096), (3, 1000), (4, 77)])
def test_objective_never_increases_and_centroids_ascend(oracle, seed, m, round_fp32):
    x, g = _row(seed, m)
    for b in (1, 2, 3, 4):
        r = oracle.kmeans_row(x, g, 1 << b, 30, round_fp32=round_fp32, want_trace=True)
        tr = r["trace"]
        # rounding a centroid to binary32 moves the objective by at most G * (ulp/2)^2,
        # 1e-9 of the objective is far above that and far below any real increase
        assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-9)), (b, tr)
        assert np.all(np.diff(r["c"]) >= 0)
        assert r["err"] == pytest.approx(tr[-1], rel=1e-12)
        assert tr[-1] < tr[0]


def _exact_kmeans_dp(x, g, k):
    """Optimal weighted 1-D k-means cost: clusters are intervals of the sorted row."""
    order = np.argsort(x, kind="stable")
    xs, gs = x[order], g[order]
    m = len(xs)
    p0 = np.concatenate([[0.0], np.cumsum(gs)])
    p1 = np.concatenate([[0.0], np.cumsum(gs * xs)])
    p2 = np.concatenate([[0.0], np.cumsum(gs * xs * xs)])

    def cost(a, b):  # elements a..b-1
        s0 = p0[b] - p0[a]
        if s0 <= 0:
            return 0.0
        s1 = p1[b] - p1[a]
        return max(p2[b] - p2[a] - s1 * s1 / s0, 0.0)

    best = np.full((k + 1, m + 1), np.inf)
    best[0, 0] = 0.0
    for kk in range(1, k + 1):
        for b in range(1, m + 1):
            for a in range(kk - 1, b):
                v = best[kk - 1, a] + cost(a, b)
                if v < best[kk, b]:
                    best[kk, b] = v
    return min(best[kk, m] for kk in range(1, k + 1))


def _brute_two_clusters(x, g):
    order = np.argsort(x, kind="stable")
    xs, gs = x[order], g[order]
    best = np.inf
    for cut in range(1, len(xs)):
        e = 0.0
        for part_x, part_g in ((xs[:cut], gs[:cut]), (xs[cut:], gs[cut:])):
            c = np.sum(part_g * part_x) / np.sum(part_g)
            e += np.sum(part_g * (part_x - c) ** 2)
        best = min(best, e)
    return best


@pytest.mark.parametrize("seed", range(6))
def test_lloyd_is_never_better_than_the_exact_optimum(oracle, seed):
    x, g = _row(100 + seed, 40, outliers=0.05)
    scale = max(np.sum(g * x * x), 1e-30)
    assert _exact_kmeans_dp(x, g, 2) == pytest.approx(_brute_two_clusters(x, g), rel=1e-9)
    for b in (1, 2, 3, 4):
        opt = _exact_kmeans_dp(x, g, 1 << b)
        r = oracle.kmeans_row(x, g, 1 << b, 50, round_fp32=False)
        assert r["err"] >= opt - 1e-12 * scale


@pytest.mark.parametrize("seed,m,b", [(7, 300, 2), (8, 2048, 3), (9, 2048, 4), (10, 999, 1)])
def test_converged_result_is_a_fixed_point(oracle, seed, m, b):
    """At convergence every centroid is the weighted mean of its members and every element
    sits with its nearest centroid (checked with numpy, not with the oracle's own loops)."""
    x, g = _row(seed, m)
    k = 1 << b
    r = oracle.kmeans_row(x, g, k, 400, round_fp32=False, want_trace=True)
    assert r["trace"][-1] == r["trace"][-5], "not converged in 400 iterations"
    lab, c = r["label"], r["c"]
    for j in range(k):
        sel = lab == j
        if sel.any():
            assert c[j] == pytest.approx(np.sum(g[sel] * x[sel]) / np.sum(g[sel]), rel=1e-12)
    np.testing.assert_array_equal(lab, np.argmin(np.abs(x[:, None] - c[None, :]), axis=1))
    assert r["err"] == pytest.approx(np.sum(g * (x - c[lab]) ** 2), rel=1e-12)


@pytest.mark.parametrize("weighted", [False, True])
@pytest.mark.parametrize("seed,m,b,iters", [(11, 600, 2, 7), (12, 1500, 3, 12), (13, 3000, 4, 20)])
def test_matches_library_kmeans_given_the_same_init(oracle, seed, m, b, iters, weighted):
    """scikit-learn's Lloyd K-means with our explicit init, one run, a fixed number of
    iterations and sample weights is the textbook weighted K-means; uniform weights give the
    unweighted special case."""
    sk = pytest.importorskip("sklearn.cluster")
    x, g = _row(seed, m)
    if not weighted:
        g = np.ones_like(x)
    k = 1 << b
    srt = np.sort(x)
    init = np.array([srt[((2 * j + 1) * m) // (2 * k)] for j in range(k)])
    km = sk.KMeans(n_clusters=k, init=init.reshape(-1, 1), n_init=1, max_iter=iters, tol=0.0,
                   algorithm="lloyd")
    import warnings
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        km.fit(x.reshape(-1, 1), sample_weight=g)
    r = oracle.kmeans_row(x, g, k, iters, round_fp32=False)
    ref = np.sort(km.cluster_centers_.ravel())
    np.testing.assert_allclose(r["c"], ref, rtol=1e-9, atol=1e-12)
    assert r["err"] == pytest.approx(np.sum(g * (x - ref[km.labels_ if np.all(np.diff(
        km.cluster_centers_.ravel()) > 0) else np.argmin(np.abs(x[:, None] - ref[None, :]), axis=1)]) ** 2),
        rel=1e-9)


def test_two_point_masses(oracle):
    # two separated clumps: the two centroids are the clumps' weighted means
    x = np.array([-1.0, -1.25, -0.75, 2.0, 2.5, 3.0, 2.25])
    g = np.array([1.0, 2.0, 1.0, 4.0, 1.0, 1.0, 2.0])
    r = oracle.kmeans_row(x, g, 2, 10, round_fp32=False)
    np.testing.assert_allclose(r["c"], [np.sum(g[:3] * x[:3]) / 4.0, np.sum(g[3:] * x[3:]) / 8.0], rtol=1e-15)


@pytest.mark.parametrize("b", [1, 2, 3, 4])
def test_zero_error_when_few_distinct_values(oracle, b):
    k = 1 << b
    rng = np.random.default_rng(5)
    for D in range(1, k + 1):
        vals = np.sort(rng.standard_normal(D)).astype(np.float16).astype(np.float64)
        vals = np.unique(vals)
        x = rng.choice(vals, size=200)
        x[:len(vals)] = vals
        g = rng.lognormal(0, 1, size=200)
        r = oracle.kmeans_row(x, g, k, 30)
        assert r["err"] == 0.0
        np.testing.assert_array_equal(r["c"][:len(vals)], vals)
        np.testing.assert_array_equal(r["c"][len(vals):], vals[-1])
        np.testing.assert_array_equal(vals[r["label"]], x)
    # the quantile init alone would not give zero error here: 1000 zeros and three other values
    x = np.array([0.0] * 1000 + [1.0, 2.0, 3.0])
    r = oracle.kmeans_row(x, np.ones_like(x), 4, 30)
    assert r["err"] == 0.0 and list(r["c"]) == [0.0, 1.0, 2.0, 3.0]


def test_exact_power_of_two_symmetries(oracle):
    w, g = inputs.make_rows(4, 1024, 21)
    base = oracle.cluster_rows(w, g, [1, 2, 3, 4], 20)
    # values * 2^p: centroids * 2^p, err * 4^p, same labels
    up = oracle.cluster_rows((w.astype(np.float32) * 8).astype(np.float16), g, [1, 2, 3, 4], 20)
    np.testing.assert_array_equal(up["centroids"], base["centroids"] * 8)
    np.testing.assert_allclose(up["err"], base["err"] * 64, rtol=1e-14)
    np.testing.assert_array_equal(up["codes"], base["codes"])
    # importance * 2^p: same centroids and labels, err * 2^p
    gi = oracle.cluster_rows(w, g * np.float32(0.25), [1, 2, 3, 4], 20)
    np.testing.assert_array_equal(gi["centroids"], base["centroids"])
    np.testing.assert_allclose(gi["err"], base["err"] * 0.25, rtol=1e-14)
    np.testing.assert_array_equal(gi["codes"], base["codes"])
    # a column permutation permutes the labels and nothing else (sums re-associate: 1e-12)
    perm = np.random.default_rng(3).permutation(1024)
    pm = oracle.cluster_rows(w[:, perm], g[:, perm], [1, 2, 3, 4], 20, round_fp32=False)
    b64 = oracle.cluster_rows(w, g, [1, 2, 3, 4], 20, round_fp32=False)
    np.testing.assert_allclose(pm["centroids"], b64["centroids"], rtol=1e-12)
    np.testing.assert_array_equal(pm["codes"], b64["codes"][:, :, perm])
    # a constant scale 2^p divides the centroids, keeps the labels
    sc = oracle.cluster_rows(w, g, [1, 2, 3, 4], 20, s=np.full(1024, 4.0, np.float32))
    np.testing.assert_array_equal(sc["centroids"] * 4, base["centroids"])
    np.testing.assert_array_equal(sc["codes"], base["codes"])
    np.testing.assert_allclose(sc["err"] * 16, base["err"], rtol=1e-14)


def test_labels_follow_the_midpoint_rule(oracle):
    """label = number of midpoints (c_j + c_{j+1})/2 strictly below the element, including rows
    with heavily repeated values (duplicate centroids)."""
    w, g = inputs.make_rows(6, 700, 33)
    w[1, :400] = 0.0
    w[2, :] = np.round(w[2, :].astype(np.float32) * 64).astype(np.float16) / np.float16(64)
    w[3, 100:650] = np.float16(0.0123)
    res = oracle.cluster_rows(w, g, [1, 2, 3, 4], 9)
    off = 0
    for bi, b in enumerate([1, 2, 3, 4]):
        k = 1 << b
        c = res["centroids"][:, off:off + k]
        t = 0.5 * (c[:, :-1] + c[:, 1:])
        want = (t[:, None, :] < w.astype(np.float64)[:, :, None]).sum(axis=2)
        np.testing.assert_array_equal(res["codes"][bi], want)
        assert np.all(np.diff(c, axis=1) >= 0)
        off += k


def test_scaled_rows_cluster_the_binary32_product(oracle):
    w, g = inputs.make_rows(3, 513, 41)
    s = inputs.make_scale(513, 41)
    res = oracle.cluster_rows(w, g, [2, 3], 15, s=s)
    r = np.float32(1.0) / s
    xt = (w.astype(np.float32) * r).astype(np.float32)
    for i in range(3):
        off = 0
        for bi, b in enumerate([2, 3]):
            one = oracle.kmeans_row(xt[i].astype(np.float64), g[i].astype(np.float64), 1 << b, 15)
            np.testing.assert_array_equal(res["centroids"][i, off:off + (1 << b)], one["c"])
            assert res["err"][i, bi] == one["err"]
            np.testing.assert_array_equal(res["codes"][bi, i], one["label"])
            off += 1 << b


def test_row_bits_selects_one_width_per_row(oracle):
    w, g = inputs.make_rows(5, 256, 55)
    full = oracle.cluster_rows(w, g, [1, 2, 3, 4], 10)
    bits = np.array([1, 4, 2, 3, 4], np.uint8)
    sel = oracle.cluster_rows(w, g, [1, 2, 3, 4], 10, row_bits=bits)
    offs = {1: 0, 2: 2, 3: 6, 4: 14}
    for i, b in enumerate(bits):
        o = offs[int(b)]
        np.testing.assert_array_equal(sel["centroids"][i, o:o + (1 << b)], full["centroids"][i, o:o + (1 << b)])
        assert sel["err"][i, b - 1] == full["err"][i, b - 1]
        np.testing.assert_array_equal(sel["codes"][b - 1, i], full["codes"][b - 1, i])


def test_centroids_are_binary32_values_and_close_to_binary64_run(oracle):
    w, g = inputs.make_rows(8, 2048, 77)
    a = oracle.cluster_rows(w, g, [1, 2, 3, 4], 25, round_fp32=True)
    b = oracle.cluster_rows(w, g, [1, 2, 3, 4], 25, round_fp32=False)
    np.testing.assert_array_equal(a["centroids"], a["centroids"].astype(np.float32).astype(np.float64))
    # the two runs can only part ways through a near-tie flip; on these rows they do not
    np.testing.assert_allclose(a["centroids"], b["centroids"], rtol=2e-7)
    np.testing.assert_allclose(a["err"], b["err"], rtol=1e-6)


def test_half_conversions_match_numpy(oracle):
    lib = oracle.lib()
    allh = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = allh.view(np.float16).astype(np.float32)
    got = np.array([lib.skim_oracle_half_to_float(int(h)) for h in allh], dtype=np.float32)
    fin = np.isfinite(ref)
    np.testing.assert_array_equal(got[fin].view(np.uint32), ref[fin].view(np.uint32))
    rng = np.random.default_rng(0)
    f = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(0.02),
        (rng.standard_normal(5000) * 1e-6).astype(np.float32),
        (rng.standard_normal(2000) * 3e4).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 6.1035e-5, 6.0976e-5, 5.96e-8, 2.98e-8, 2.9803e-8,
                  1.00048828125, 1.0009765625 + 2 ** -12, 2 ** -14, 2 ** -14 - 2 ** -26], np.float32)])
    with np.errstate(over="ignore"):
        want = f.astype(np.float16).view(np.uint16)
    got = np.array([lib.skim_oracle_float_to_half(float(v)) for v in f], dtype=np.uint16)
    np.testing.assert_array_equal(got, want)
