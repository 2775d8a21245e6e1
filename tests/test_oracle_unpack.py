"""Pins for the oracle's unpacking side: dequantised weights and the matrix-vector product taken
from the packed form (Section 4 overview; Section 4.2, last paragraph; Section 4.3).  CPU only."""
import numpy as np
import pytest

from paper_2412_04180_b200 import inputs


def _hand_example():
    """Two rows of five elements, worked by hand.

    Row 0 has width 2 and codes [3, 0, 1, 2, 1]: element j sits in bits [2j, 2j+2), so the set bits
    are 0, 1 (code 3), 4 (code 1), 7 (code 2) and 8 (code 1): 1 + 2 + 16 + 128 + 256 = 403.
    Row 1 has width 1 and codes [1, 0, 1, 1, 0]: bits 0, 2, 3 -> 13.
    Groups go by ascending width, so the width-1 row comes first; a row of 5 elements takes
    ceil(5 b / 32) = 1 word, rounded up to 4.
    """
    em = dict(packed=np.array([13, 0, 0, 0, 403, 0, 0, 0], np.uint32), row_order=np.array([1, 0], np.int32),
              group_start=np.array([0, 1, 2], np.int64), group_word=np.array([0, 4, 8], np.int64),
              lut=np.array([[-1.5, -0.5, 0.25, 2.0], [-1.0, 3.0, 3.0, 3.0]], np.float16).view(np.uint16))
    s = np.array([1, 2, 0.5, 4, 1], np.float32)
    x = np.array([1, -1, 2, 0.5, 4], np.float16)
    # row 0: lut[3,0,1,2,1] = [2, -1.5, -0.5, 0.25, -0.5], times s; row 1: lut[1,0,1,1,0] = [3, -1, 3, 3, -1], times s
    wq = np.array([[2, -3, -0.25, 1, -0.5], [3, -2, 1.5, 12, -1]], np.float16)
    wq_unscaled = np.array([[2, -1.5, -0.5, 0.25, -0.5], [3, -1, 3, 3, -1]], np.float16)
    # z = x * s = [1, -2, 1, 2, 4]; y0 = 2 + 3 - 0.5 + 0.5 - 2 = 3; y1 = 3 + 2 + 3 + 6 - 4 = 10
    y = np.array([3.0, 10.0])
    # without s: y0 = 2 + 1.5 - 1 + 0.125 - 2 = 0.625; y1 = 3 + 1 + 6 + 1.5 - 4 = 7.5
    y_unscaled = np.array([0.625, 7.5])
    return em, s, x, wq, wq_unscaled, y, y_unscaled


def test_hand_worked_unpacking(oracle):
    em, s, x, wq, wq_unscaled, y, y_unscaled = _hand_example()
    np.testing.assert_array_equal(oracle.dequantize(em, 5, [1, 2], s=s).view(np.uint16), wq.view(np.uint16))
    np.testing.assert_array_equal(oracle.dequantize(em, 5, [1, 2]).view(np.uint16), wq_unscaled.view(np.uint16))
    got, mag = oracle.matvec(em, 5, [1, 2], x, s=s)
    np.testing.assert_array_equal(got, y)
    np.testing.assert_array_equal(mag, [8.0, 18.0])          # sums of the absolute terms above
    got, _ = oracle.matvec(em, 5, [1, 2], x)
    np.testing.assert_array_equal(got, y_unscaled)


def _emit_case(oracle, rows, cols, seed, scaled):
    w, g = inputs.make_rows(rows, cols, seed)
    s = inputs.make_scale(cols, seed + 1) if scaled else None
    res = oracle.cluster_rows(w, g, [1, 2, 3, 4], 6, s=s)
    bits = ((np.arange(rows) * 5 + seed) % 4 + 1).astype(np.uint8)
    em = oracle.emit(w, bits, res["centroids"].astype(np.float32), [1, 2, 3, 4], s=s)
    return w, s, bits, em


@pytest.mark.parametrize("cols", [1, 7, 31, 32, 33, 100, 257, 1000])
@pytest.mark.parametrize("scaled", [False, True])
def test_dequantize_is_codebook_entry_times_scale(oracle, cols, scaled):
    """Written from the labels the packer was given (not from the packed words): numpy gathers the
    codebook entries, multiplies by the scale in binary32 and rounds to binary16."""
    rows = 19
    w, s, bits, em = _emit_case(oracle, rows, cols, 300 + cols, scaled)
    lut = em["lut"].view(np.float16).astype(np.float32)
    want = np.take_along_axis(lut, em["codes"].astype(np.int64), axis=1)
    if scaled:
        want = (want * s[None, :].astype(np.float32)).astype(np.float32)
    got = oracle.dequantize(em, cols, [1, 2, 3, 4], s=s)
    np.testing.assert_array_equal(got.view(np.uint16), want.astype(np.float16).view(np.uint16))
    # Section 4.3: the dequantised weight approximates the original one (4-bit rows closely)
    if cols >= 100:
        four = bits == 4
        err = np.abs(got[four].astype(np.float64) - w[four].astype(np.float64)).mean()
        assert err < 0.25 * np.abs(w[four].astype(np.float64)).mean()


@pytest.mark.parametrize("cols", [5, 64, 333, 1024])
@pytest.mark.parametrize("scaled", [False, True])
def test_matvec_is_the_dense_product(oracle, cols, scaled):
    rows = 23
    w, s, bits, em = _emit_case(oracle, rows, cols, 500 + cols, scaled)
    rng = np.random.default_rng(cols)
    x = rng.standard_normal(cols).astype(np.float16)
    lut = em["lut"].view(np.float16).astype(np.float64)
    dense = np.take_along_axis(lut, em["codes"].astype(np.int64), axis=1)
    z = x.astype(np.float32) * s if scaled else x.astype(np.float32)
    y, mag = oracle.matvec(em, cols, [1, 2, 3, 4], x, s=s)
    np.testing.assert_allclose(y, dense @ z.astype(np.float64), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(mag, np.abs(dense) @ np.abs(z.astype(np.float64)), rtol=1e-12)
    # a unit vector picks one column of the quantised matrix
    j = cols // 2
    e = np.zeros(cols, np.float16)
    e[j] = 1.0
    col, _ = oracle.matvec(em, cols, [1, 2, 3, 4], e, s=s)
    np.testing.assert_array_equal(col, dense[:, j] * (float(s[j]) if scaled else 1.0))
    # linearity in x (exact for power-of-two factors)
    y2, _ = oracle.matvec(em, cols, [1, 2, 3, 4], (x.astype(np.float32) * 2).astype(np.float16), s=s)
    np.testing.assert_array_equal(y2, 2 * y)
