"""Pins for the oracle's greedy allocator (Algorithm 1), code emission and scaling-vector update
(Algorithm 2).  CPU only; nothing here touches the CUDA path."""
import itertools

import numpy as np
import pytest

from paper_2412_04180_b200 import inputs


# ---------------------------------------------------------------- allocation (Algorithm 1)

def _brute_force_allocation(err, b_min, total):
    rows, nb = err.shape
    best, best_cost = None, np.inf
    for combo in itertools.product(range(nb), repeat=rows):
        if sum(combo) + rows * b_min != total:
            continue
        cost = sum(float(err[i, c]) for i, c in enumerate(combo))
        if cost < best_cost - 1e-12:
            best, best_cost = combo, cost
    return best_cost


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("budget", [1.0, 1.5, 2.2, 3.0, 3.5, 4.0])
def test_greedy_is_optimal_when_gains_do_not_increase(oracle, seed, budget):
    """With non-increasing marginal gains in every row, unit-step greedy solves the budgeted
    minimisation of Section 4.2 exactly; brute force over all 4^6 allocations confirms it."""
    rows = 6
    rng = np.random.default_rng(seed)
    gains = np.sort(rng.integers(1, 40, size=(rows, 3)), axis=1)[:, ::-1].astype(np.float64)
    tail = rng.integers(1, 5, size=(rows, 1)).astype(np.float64)
    err = np.concatenate([gains, tail], axis=1)[:, ::-1].cumsum(axis=1)[:, ::-1].astype(np.float32)
    bits, total = oracle.allocate_bits(err, 1, budget)
    assert total == int(np.floor(rows * budget + 1e-6))
    assert int(bits.sum()) == total
    assert bits.min() >= 1 and bits.max() <= 4
    cost = sum(float(err[i, b - 1]) for i, b in enumerate(bits))
    assert cost == pytest.approx(_brute_force_allocation(err, 1, total), abs=1e-9)


def test_allocation_budget_rounding_and_limits(oracle):
    err = inputs.make_error_table(256, 4, 3)
    bits, total = oracle.allocate_bits(err, 1, 3.2)
    assert total == 819 and bits.sum() == 819            # 256 * 3.2 = 819.2 -> 819
    bits, total = oracle.allocate_bits(err, 1, 3.0)
    assert total == 768 and bits.sum() == 768             # average equals the budget exactly
    bits, _ = oracle.allocate_bits(err, 1, 1.0)
    assert np.all(bits == 1)
    bits, _ = oracle.allocate_bits(err, 1, 4.0)
    assert np.all(bits == 4)
    with pytest.raises(ValueError):
        oracle.allocate_bits(err, 1, 0.9)
    with pytest.raises(ValueError):
        oracle.allocate_bits(err, 1, 4.1)


def test_allocation_hand_example(oracle):
    # gains: row0 (10, 1, 1)  row1 (4, 3, 2)  row2 (4, 5, 0): row 2's second bit is worth more
    # than its first.  Sequence by Algorithm 1 (largest gain, lowest row on ties):
    # row0 (10), row1 (4, tie with row2 -> lower row), row2 (4), row2 (5), row1 (3), row1 (2) ...
    err = np.array([[12, 2, 1, 0], [9, 5, 2, 0], [9, 5, 0, 0]], np.float32)
    expect = {3: [1, 1, 1], 4: [2, 1, 1], 5: [2, 2, 1], 6: [2, 2, 2], 7: [2, 2, 3], 8: [2, 3, 3], 9: [2, 4, 3]}
    for total, want in expect.items():
        bits, tot = oracle.allocate_bits(err, 1, total / 3.0)
        assert tot == total
        assert list(bits) == want, total


def test_allocation_takes_negative_gains_when_the_budget_demands_it(oracle):
    err = np.array([[1, 2, 3, 4], [5, 1, 2, 9]], np.float32)   # more bits make it worse
    bits, total = oracle.allocate_bits(err, 1, 4.0)
    assert list(bits) == [4, 4] and total == 8
    bits, _ = oracle.allocate_bits(err, 1, 1.5)
    assert list(bits) == [1, 2]


def _brute_force_from(err, b_min, start, total):
    """Cheapest allocation with every width >= start and the given total."""
    rows, nb = err.shape
    best = np.inf
    for combo in itertools.product(range(start - b_min, nb), repeat=rows):
        if sum(combo) + rows * b_min != total:
            continue
        best = min(best, sum(float(err[i, c]) for i, c in enumerate(combo)))
    return best


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("budget", [1.0, 1.5, 2.0, 2.4, 3.0, 3.7, 4.0])
def test_floor_started_allocation(oracle, seed, budget):
    """Every row starts at floor(budget): an integer budget switches mixed precision off; otherwise the
    remaining bits go greedily, which on tables with non-increasing gains is the optimum among the
    allocations that give every row at least floor(budget) bits (brute force)."""
    rows = 6
    rng = np.random.default_rng(100 + seed)
    gains = np.sort(rng.integers(1, 40, size=(rows, 3)), axis=1)[:, ::-1].astype(np.float64)
    tail = rng.integers(1, 5, size=(rows, 1)).astype(np.float64)
    err = np.concatenate([gains, tail], axis=1)[:, ::-1].cumsum(axis=1)[:, ::-1].astype(np.float32)
    bits, total = oracle.allocate_bits(err, 1, budget, floor_start=True)
    start = int(np.floor(budget + 1e-9))
    assert total == int(np.floor(rows * budget + 1e-6)) and int(bits.sum()) == total
    assert bits.min() >= start and bits.max() <= 4
    if budget == start:
        assert np.all(bits == start)
    cost = sum(float(err[i, b - 1]) for i, b in enumerate(bits))
    assert cost == pytest.approx(_brute_force_from(err, 1, start, total), abs=1e-9)
    # never cheaper than the unconstrained greedy, which may leave rows below the floor
    free, _ = oracle.allocate_bits(err, 1, budget)
    assert cost >= sum(float(err[i, b - 1]) for i, b in enumerate(free)) - 1e-9


def test_floor_started_allocation_hand_example(oracle):
    # budget 7/3 = 2.33: every row starts at 2 bits, one bit is left: the gains of the third bit are
    # 1 (row 0), 3 (row 1), 5 (row 2) -> row 2.  The plain greedy from 1 bit gives [2, 2, 3] as well here;
    # at budget 5/3 the floor is 1 and both agree by definition.
    err = np.array([[12, 2, 1, 0], [9, 5, 2, 0], [9, 5, 0, 0]], np.float32)
    bits, total = oracle.allocate_bits(err, 1, 7 / 3, floor_start=True)
    assert total == 7 and list(bits) == [2, 2, 3]
    # a table where the floor matters: row 0 gains nothing from its second bit, the plain greedy leaves it at 1
    err = np.array([[5, 5, 5, 5], [9, 4, 1, 0], [9, 4, 1, 0]], np.float32)
    plain, _ = oracle.allocate_bits(err, 1, 2.0)
    floor, _ = oracle.allocate_bits(err, 1, 2.0, floor_start=True)
    assert list(plain) == [1, 3, 2] and list(floor) == [2, 2, 2]


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("budget", [1.0, 1.5, 2.2, 3.0, 3.5, 4.0])
def test_optimal_allocation_is_the_brute_force_minimum(oracle, seed, budget):
    """The dynamic programme against brute force over all 4^6 allocations, on tables whose gains go up and
    down (where the greedy need not be optimal), and against the greedy itself."""
    rows = 6
    rng = np.random.default_rng(200 + seed)
    err = rng.integers(0, 50, size=(rows, 4)).astype(np.float32)
    bits, total, cost = oracle.allocate_optimal(err, 1, budget)
    assert total == int(np.floor(rows * budget + 1e-6)) and int(bits.sum()) == total
    assert bits.min() >= 1 and bits.max() <= 4
    assert cost == sum(float(err[i, b - 1]) for i, b in enumerate(bits))
    assert cost == pytest.approx(_brute_force_allocation(err, 1, total), abs=1e-9)
    greedy, _ = oracle.allocate_bits(err, 1, budget)
    assert cost <= sum(float(err[i, b - 1]) for i, b in enumerate(greedy)) + 1e-9


def test_optimal_allocation_equals_greedy_cost_when_gains_do_not_increase(oracle):
    rows = 300
    rng = np.random.default_rng(7)
    gains = np.sort(rng.integers(1, 1000, size=(rows, 3)), axis=1)[:, ::-1].astype(np.float64)
    err = np.concatenate([gains, np.ones((rows, 1))], axis=1)[:, ::-1].cumsum(axis=1)[:, ::-1].astype(np.float32)
    for budget in (1.0, 1.7, 2.5, 3.0, 3.9, 4.0):
        bits, total, cost = oracle.allocate_optimal(err, 1, budget)
        greedy, gtotal = oracle.allocate_bits(err, 1, budget)
        assert total == gtotal
        assert cost == sum(float(err[i, b - 1]) for i, b in enumerate(greedy))     # integers: exact


def test_allocation_with_the_printed_stopping_rule(oracle):
    """Algorithm 1 as printed stops once the total reaches rows * budget: restated here as a plain Python loop."""
    rng = np.random.default_rng(11)
    err = rng.integers(0, 60, size=(37, 4)).astype(np.float32)
    for budget in (1.0, 1.01, 2.5, 3.2, 3.99, 4.0):
        bits = [1] * 37
        while sum(bits) < 37 * budget - 1e-6:
            gains = [(float(err[i, b - 1]) - float(err[i, b]), -i) for i, b in enumerate(bits) if b < 4]
            rows_left = [i for i, b in enumerate(bits) if b < 4]
            best = max(range(len(gains)), key=lambda q: gains[q])
            bits[rows_left[best]] += 1
        got, total = oracle.allocate_bits(err, 1, budget, round_up=True)
        assert list(got) == bits and total == sum(bits)
        assert total == int(np.ceil(37 * budget - 1e-6))
        down, tdown = oracle.allocate_bits(err, 1, budget)
        assert tdown <= total <= tdown + 1


# ---------------------------------------------------------------- emission

def _unpack_row(words, cols, b):
    bits = np.unpackbits(words.view(np.uint8), bitorder="little")[:cols * b].reshape(cols, b)
    return (bits * (1 << np.arange(b))).sum(axis=1).astype(np.uint8)


@pytest.mark.parametrize("cols", [1, 31, 32, 33, 127, 512, 1000])
def test_pack_unpack_round_trip_and_layout(oracle, cols):
    rows = 23
    w, g = inputs.make_rows(rows, cols, 60 + cols)
    s = inputs.make_scale(cols, 9)
    res = oracle.cluster_rows(w, g, [1, 2, 3, 4], 8, s=s)
    bits = (np.arange(rows) * 7 % 4 + 1).astype(np.uint8)
    cent = res["centroids"].astype(np.float32)
    em = oracle.emit(w, bits, cent, [1, 2, 3, 4], s=s)
    # groups: ascending width, ascending row inside a group
    want_order = sorted(range(rows), key=lambda i: (bits[i], i))
    assert list(em["row_order"]) == want_order
    offs = {1: 0, 2: 2, 3: 6, 4: 14}
    word = 0
    for bi, b in enumerate([1, 2, 3, 4]):
        stride = oracle.row_stride_words(cols, b)
        assert stride % 4 == 0 and stride * 32 >= cols * b and (stride - 4) * 32 < cols * b
        assert em["group_word"][bi] == word
        for p in range(int(em["group_start"][bi]), int(em["group_start"][bi + 1])):
            i = em["row_order"][p]
            assert bits[i] == b
            row_words = em["packed"][word:word + stride]
            codes = _unpack_row(row_words, cols, b)
            # the packed labels are the clustering's own final labels
            np.testing.assert_array_equal(codes, res["codes"][bi, i])
            np.testing.assert_array_equal(codes, em["codes"][i])
            # padding is zero
            tail = np.unpackbits(row_words.view(np.uint8), bitorder="little")[cols * b:]
            assert not tail.any()
            # LUT: binary16 round-to-nearest of the centroids, padded with the last entry
            k = 1 << b
            c = cent[i, offs[b]:offs[b] + k]
            lut = em["lut"][i].view(np.float16)
            np.testing.assert_array_equal(lut[:k].view(np.uint16), c.astype(np.float16).view(np.uint16))
            np.testing.assert_array_equal(lut[k:].view(np.uint16), np.full(16 - k, lut[k - 1]).view(np.uint16))
            word += stride
    assert em["group_word"][4] == word == len(em["packed"])


def test_dequantised_matrix_is_lut_times_scale(oracle):
    """Section 4.3: Wq = replace(c, L) * alpha; the reconstruction error it gives equals the
    clustering's err up to the binary16 rounding of the centroids."""
    rows, cols = 12, 640
    w, g = inputs.make_rows(rows, cols, 71)
    s = np.full(cols, 2.0, np.float32)
    res = oracle.cluster_rows(w, g, [1, 2, 3, 4], 20, s=s)
    bits = np.array([4] * rows, np.uint8)
    em = oracle.emit(w, bits, res["centroids"].astype(np.float32), [1, 2, 3, 4], s=s)
    lut = em["lut"].view(np.float16).astype(np.float64)
    wq = np.take_along_axis(lut, em["codes"].astype(np.int64), axis=1) * s.astype(np.float64)
    rec = (g.astype(np.float64) * (w.astype(np.float64) - wq) ** 2).sum(axis=1)
    # err is measured on the scaled values x~ = w / 2, so in w units it is 4x
    np.testing.assert_allclose(rec, 4.0 * res["err"][:, 3], rtol=2e-2)


# ---------------------------------------------------------------- scaling vector (Algorithm 2)

def _numpy_loss(w, g, labels, alpha):
    """loss(alpha) written from the definition, independently of the oracle's loops."""
    w = w.astype(np.float64)
    g = g.astype(np.float64)
    total = 0.0
    for i in range(w.shape[0]):
        for k in np.unique(labels[i]):
            sel = labels[i] == k
            gk = g[i, sel]
            c = np.sum(gk * w[i, sel] / alpha[sel]) / np.sum(gk)
            total += np.sum(gk * (w[i, sel] - alpha[sel] * c) ** 2)
    return total


def test_scale_loss_and_gradient(oracle):
    rows, cols = 9, 48
    w, g = inputs.make_rows(rows, cols, 81, outlier_frac=0.02)
    res = oracle.cluster_rows(w, g, [2], 10)
    labels = res["codes"][0]
    alpha = inputs.make_scale(cols, 5, spread=0.1).astype(np.float64)
    loss, grad = oracle.scale_loss_grad(w, g, labels, alpha)
    assert loss == pytest.approx(_numpy_loss(w, g, labels, alpha), rel=1e-12)
    # at alpha = 1 the loss is the K-means objective of the fixed labels with re-fitted centroids
    loss1, _ = oracle.scale_loss_grad(w, g, labels, np.ones(cols))
    assert loss1 <= res["err"][:, 0].sum() * (1 + 1e-6)
    # central finite differences of the independently written loss
    for j in range(0, cols, 5):
        h = 1e-6
        ap, am = alpha.copy(), alpha.copy()
        ap[j] += h
        am[j] -= h
        fd = (_numpy_loss(w, g, labels, ap) - _numpy_loss(w, g, labels, am)) / (2 * h)
        assert grad[j] == pytest.approx(fd, rel=2e-5, abs=1e-9 * np.abs(grad).max())


def test_adam_schedule_and_descent(oracle):
    rows, cols = 16, 64
    w, g = inputs.make_rows(rows, cols, 91, outlier_frac=0.02)
    labels = oracle.cluster_rows(w, g, [2], 10)["codes"][0]
    a0 = np.ones(cols)
    a1, tr = oracle.scale_update(w, g, labels, a0, steps=1)
    # the first Adam step moves every coordinate by lr * sign(grad) (bias-corrected, eps tiny)
    _, grad = oracle.scale_loss_grad(w, g, labels, a0)
    np.testing.assert_allclose(a1 - a0, -0.01 * grad / (np.abs(grad) + 1e-8), rtol=1e-9, atol=1e-15)
    # steps 40..79 run at half the rate, 80..119 at a quarter: replay Adam in numpy
    alpha, m1, m2 = a0.copy(), np.zeros(cols), np.zeros(cols)
    for t in range(90):
        _, gr = oracle.scale_loss_grad(w, g, labels, alpha)
        m1 = 0.9 * m1 + 0.1 * gr
        m2 = 0.999 * m2 + 0.001 * gr * gr
        lr = 0.01 * 0.5 ** (t // 40)
        alpha = alpha - lr * (m1 / (1 - 0.9 ** (t + 1))) / (np.sqrt(m2 / (1 - 0.999 ** (t + 1))) + 1e-8)
    a90, tr90 = oracle.scale_update(w, g, labels, a0, steps=90)
    np.testing.assert_allclose(a90, alpha, rtol=1e-10)
    # training the scale lowers the reconstruction loss
    a120, tr120 = oracle.scale_update(w, g, labels, a0, steps=120)
    final, _ = oracle.scale_loss_grad(w, g, labels, a120, want_grad=False)
    assert final < tr120[0]
