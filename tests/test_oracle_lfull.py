"""Pins of the oracle's L-full error and residual (Section 3.4; Section 4.2; Algorithm 3), none of which
involves the CUDA path: a hand-worked example, equality with |d X|^2 formed explicitly, the diagonal
special case (the paper's L-diag / S-diag forms) against the K-means oracle's own error, exact symmetries."""
import os

import numpy as np
import pytest

from paper_2412_04180_b200 import inputs

BITS = [1, 2, 3, 4]
HERE = os.path.dirname(os.path.abspath(__file__))


def test_hand_example(oracle):
    text = open(os.path.join(HERE, "golden", "lfull_hand_example.txt")).read().splitlines()
    rows = {}
    for line in text:
        if line.startswith("#") or not line.strip():
            continue
        name, rest = line.split(":")
        rows[name.strip()] = rest
    H = np.array([[float(v) for v in r.split()] for r in rows["H"].split(";")], dtype=np.float16)
    for name in "ABC":
        d, want = rows[name].split("->")
        d = np.array([float(v) for v in d.split()], dtype=np.float64)
        for e in (0, 3):
            D = (d * 2.0 ** e).astype(np.float16)[None, :]
            err, mag = oracle.err_lfull(D, H, exp2=e)
            assert err[0] == float(want)
            assert mag[0] >= err[0]


def test_equals_squared_norm_of_d_times_x(oracle):
    """H = X X^T with X in {-1, 0, 1}: H is integer, exact in binary16, and d H d^T = |d X|^2."""
    rng = np.random.default_rng(3)
    cols, samples, rows = 150, 40, 9
    X = rng.integers(-1, 2, size=(cols, samples)).astype(np.float64)
    H = (X @ X.T).astype(np.float16)
    assert np.array_equal(H.astype(np.float64), X @ X.T)
    D = (rng.standard_normal((rows, cols)) * 3).astype(np.float16)
    err, _ = oracle.err_lfull(D, H, exp2=0)
    want = ((D.astype(np.float64) @ X) ** 2).sum(axis=1)
    np.testing.assert_allclose(err, want, rtol=1e-12)
    # the quadratic form does not see the antisymmetric part of H, and scales exactly with powers of two
    Hn = H.copy()
    Hn[3, 7] = np.float16(float(H[3, 7]) + 2)
    Hn[7, 3] = np.float16(float(H[7, 3]) - 2)
    np.testing.assert_allclose(oracle.err_lfull(D, Hn, exp2=0)[0], err, rtol=1e-12)
    e2, m2 = oracle.err_lfull((D.astype(np.float32) * 4).astype(np.float16), H, exp2=2)
    np.testing.assert_array_equal(e2, err)
    np.testing.assert_array_equal(oracle.err_lfull(D, (H.astype(np.float32) * 2).astype(np.float16), exp2=0)[0], 2 * err)


def test_diagonal_h_gives_the_clustering_error(oracle):
    """With H = diag(h) the L-full error is sum_j h_j (w_j - wq_j)^2: the paper's diagonal forms.  Clustering
    with importance h (constant down each column) records exactly that error, from its own assignment and
    its own sums; the two agree up to the binary16 rounding of the residual (2^-11 per element)."""
    rows, cols = 12, 400
    w, _ = inputs.make_rows(rows, cols, 21)
    h = np.exp(np.random.default_rng(5).standard_normal(cols)).astype(np.float16)
    g = np.tile(h.astype(np.float32), (rows, 1))
    res = oracle.cluster_rows(w, g, BITS, 20)
    H = np.diag(h.astype(np.float64)).astype(np.float16)
    for bi, b in enumerate(BITS):
        D = oracle.residual(w, res["centroids"].astype(np.float32), BITS, width=b, exp2=8)
        err, mag = oracle.err_lfull(D, H, exp2=8)
        np.testing.assert_allclose(err, res["err"][:, bi], rtol=2.0 ** -9)
        np.testing.assert_allclose(mag, err, rtol=1e-12)         # a diagonal form has no cancellation


def test_residual_against_numpy_from_the_labels(oracle):
    """d = binary16((float(w) - c[label] * alpha) * 2^e), with the labels the K-means oracle reported and
    numpy's own binary32 arithmetic and binary16 cast; zero when the row's values all have a centroid."""
    rows, cols = 10, 333
    w, g = inputs.make_rows(rows, cols, 23)
    w[4, :] = (np.arange(cols) % 7).astype(np.float16) / 16        # 7 distinct values: exact from 3 bits on
    s = inputs.make_scale(cols, 9)
    for scale in (None, s):
        res = oracle.cluster_rows(w, g, BITS, 15, s=scale)
        c32 = res["centroids"].astype(np.float32)
        off = 0
        for bi, b in enumerate(BITS):
            k = 1 << b
            D = oracle.residual(w, c32, BITS, width=b, s=scale, exp2=6)
            lab = res["codes"][bi].astype(np.int64)
            cq = np.take_along_axis(c32[:, off:off + k], lab, axis=1)
            q = cq if scale is None else (cq * scale[None, :]).astype(np.float32)
            want = ((w.astype(np.float32) - q).astype(np.float32) * np.float32(64.0)).astype(np.float16)
            np.testing.assert_array_equal(D.view(np.uint16), want.view(np.uint16))
            if b >= 3 and scale is None:
                assert not D[4].any()
            off += k
    # rows at their own widths
    bits = (np.arange(rows) % 4 + 1).astype(np.uint8)
    res = oracle.cluster_rows(w, g, BITS, 15)
    c32 = res["centroids"].astype(np.float32)
    Dr = oracle.residual(w, c32, BITS, row_bits=bits, exp2=6)
    for i, b in enumerate(bits):
        np.testing.assert_array_equal(Dr[i].view(np.uint16), oracle.residual(w, c32, BITS, width=int(b), exp2=6)[i].view(np.uint16))


def test_lfull_error_decreases_with_the_width_on_the_synthetic_gram(oracle):
    """Sanity of the synthetic H (inputs.make_gram): symmetric, positive diagonal, and finer codebooks lower
    the L-full error of almost every row although the clustering optimises the diagonal objective."""
    rows, cols = 16, 256
    w, g = inputs.make_rows(rows, cols, 29)
    H = inputs.make_gram(cols, 31)
    assert np.array_equal(H, H.T) and np.all(np.diag(H) > 0)
    res = oracle.cluster_rows(w, g, BITS, 20)
    c32 = res["centroids"].astype(np.float32)
    table = np.stack([oracle.err_lfull(oracle.residual(w, c32, BITS, width=b), H)[0] for b in BITS], axis=1)
    assert np.all(table >= 0)
    assert np.mean(table[:, 0] > table[:, 3]) == 1.0


def _labels_for(oracle, w, g, bits):
    res = oracle.cluster_rows(w, g, BITS, 15, row_bits=bits)
    return np.stack([res["codes"][int(b) - 1, i] for i, b in enumerate(bits)]).astype(np.uint8)


def test_scale_lfull_gradient_equals_finite_differences(oracle):
    """The analytic gradient of the L-full loss of the scaling vector (both terms: the explicit alpha and the
    re-fitted centroids) against central differences of the loss itself, on exact residuals."""
    rows, cols = 6, 40
    w, g = inputs.make_rows(rows, cols, 71, outlier_frac=0.02)
    bits = (np.arange(rows) % 4 + 1).astype(np.uint8)
    labels = _labels_for(oracle, w, g, bits)
    H = inputs.make_gram(cols, 72)
    alpha = inputs.make_scale(cols, 73, spread=0.1).astype(np.float64)
    loss, grad = oracle.scale_loss_grad_lfull(w, g, labels, alpha, H, round_d=False)
    # the loss itself, independently: rows of D from numpy, quadratic form by matrix products
    x = w.astype(np.float64)
    D = np.zeros_like(x)
    for i in range(rows):
        for k in range(16):
            sel = labels[i] == k
            if sel.any() and g[i, sel].sum() > 0:
                c = np.sum(g[i, sel] * x[i, sel] / alpha[sel]) / np.sum(g[i, sel].astype(np.float64))
                D[i, sel] = x[i, sel] - alpha[sel] * c
    Hd = H.astype(np.float64)
    assert loss == pytest.approx(np.einsum("ij,jk,ik->", D, Hd, D), rel=1e-12)
    for j in (0, 7, 19, 39):
        h = 1e-6 * alpha[j]
        ap, am = alpha.copy(), alpha.copy()
        ap[j] += h
        am[j] -= h
        fd = (oracle.scale_loss_grad_lfull(w, g, labels, ap, H, round_d=False, want_grad=False)[0]
              - oracle.scale_loss_grad_lfull(w, g, labels, am, H, round_d=False, want_grad=False)[0]) / (2 * h)
        assert grad[j] == pytest.approx(fd, rel=2e-5, abs=1e-9 * np.abs(grad).max())


def test_scale_lfull_with_diagonal_h_is_the_diagonal_update(oracle):
    """H = diag(h) and importance h down every column: the L-full loss of the scaling vector IS the diagonal one,
    so loss trace and alpha of the two oracle routines agree step for step."""
    rows, cols, steps = 10, 96, 25
    w, _ = inputs.make_rows(rows, cols, 81)
    h = np.exp(0.5 * np.random.default_rng(82).standard_normal(cols)).astype(np.float16)
    g = np.tile(h.astype(np.float32), (rows, 1))
    bits = (np.arange(rows) % 4 + 1).astype(np.uint8)
    labels = _labels_for(oracle, w, g, bits)
    H = np.diag(h.astype(np.float64)).astype(np.float16)
    a0 = np.ones(cols)
    a_diag, t_diag = oracle.scale_update(w, g, labels, a0, steps=steps)
    a_full, t_full = oracle.scale_update_lfull(w, g, labels, a0, H, steps=steps, round_d=False)
    np.testing.assert_allclose(t_full, t_diag, rtol=1e-10)
    np.testing.assert_allclose(a_full, a_diag, rtol=1e-9)
    # with the binary16 residual operand the loss moves by its rounding (2^-11 per element) and no more
    _, t_round = oracle.scale_update_lfull(w, g, labels, a0, H, steps=steps, round_d=True)
    np.testing.assert_allclose(t_round, t_diag, rtol=2e-3)


def test_scale_lfull_training_lowers_the_loss(oracle):
    rows, cols = 24, 64
    w, g = inputs.make_rows(rows, cols, 91)
    bits = np.full(rows, 3, np.uint8)
    labels = _labels_for(oracle, w, g, bits)
    H = inputs.make_gram(cols, 92)
    _, trace = oracle.scale_update_lfull(w, g, labels, np.ones(cols), H, steps=40)
    assert trace[-1] < trace[0]
