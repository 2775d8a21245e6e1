"""Comparison helpers for the GPU-vs-oracle parity tests.

Tolerances (the ones the path is specified with): centroids 1e-4 relative, err 1e-5 relative,
at least 99.9 % of the labels equal and every disagreement at a midpoint tie; allocation, packed
codes, row order, group tables and LUTs bit-exact when both sides get the same inputs.
"""
import numpy as np

CENT_RTOL = 1e-4
ERR_RTOL = 1e-5
LABEL_AGREE = 0.999
OFFS = {1: 0, 2: 2, 3: 6, 4: 14}


def offsets(bit_set):
    out, off = {}, 0
    for b in bit_set:
        out[int(b)] = off
        off += 1 << int(b)
    return out


def check_cluster(ora, cent, err, codes, x_values, bit_set, rows=None, label=""):
    """ora: oracle.cluster_rows result (for the same rows).  cent/err/codes: numpy from the GPU.
    x_values: float64 [rows, cols], the values that were clustered (for the tie check)."""
    oc = ora["centroids"]
    if rows is not None:
        cent, err = cent[rows], err[rows]
        if codes is not None:
            codes = codes[:, rows]
    scale = np.abs(oc).max(axis=1, keepdims=True)
    # centroids: relative to the value itself, with a floor for centroids next to zero
    tol = CENT_RTOL * np.maximum(np.abs(oc), 1e-3 * scale)
    bad = np.abs(cent.astype(np.float64) - oc) > tol
    assert not bad.any(), f"{label}: {bad.sum()} centroids differ, rows {np.unique(np.nonzero(bad)[0])[:10]}"
    np.testing.assert_allclose(err.astype(np.float64), ora["err"], rtol=ERR_RTOL, atol=1e-30, err_msg=label)
    exact = float(np.mean(cent.astype(np.float64) == oc))
    if codes is not None:
        agree = float(np.mean(codes == ora["codes"]))
        assert agree >= LABEL_AGREE, f"{label}: labels agree {agree}"
        offs = offsets(bit_set)
        for bi, b in enumerate(bit_set):
            d = np.nonzero(codes[bi] != ora["codes"][bi])
            if len(d[0]) == 0:
                continue
            # a disagreement must sit at a midpoint of either side's centroids (a tie)
            k = 1 << int(b)
            for i, j in zip(*d):
                x = x_values[i, j]
                lo, hi = sorted((int(codes[bi][i, j]), int(ora["codes"][bi][i, j])))
                assert hi == lo + 1, f"{label}: labels differ by more than one cluster"
                for c in (cent[i, offs[int(b)]:offs[int(b)] + k].astype(np.float64), oc[i, offs[int(b)]:offs[int(b)] + k]):
                    t = 0.5 * (c[lo] + c[hi])
                    if abs(x - t) <= 4 * np.spacing(np.float32(abs(t))):
                        break
                else:
                    raise AssertionError(f"{label}: label mismatch away from a midpoint (row {i}, col {j})")
    return exact


def check_cluster_at(ora, cent, err, codes, x_values, row_bits, bit_set, label=""):
    """As check_cluster, for rows clustered only at their allocated width (skim_cluster_rows_at):
    ora is oracle.cluster_rows(..., row_bits=row_bits); cent [rows, sumk], err [rows], codes [rows, cols]
    from the GPU.  Centroids, error and labels of every row's own width block are compared."""
    offs = offsets(bit_set)
    bidx = {int(b): i for i, b in enumerate(bit_set)}
    exact, total = 0, 0
    for i, b in enumerate(row_bits):
        b = int(b)
        o, k, bi = offs[b], 1 << b, bidx[b]
        oc = ora["centroids"][i, o:o + k]
        gc = cent[i, o:o + k].astype(np.float64)
        tol = CENT_RTOL * np.maximum(np.abs(oc), 1e-3 * np.abs(oc).max())
        assert np.all(np.abs(gc - oc) <= tol), f"{label}: row {i} (width {b}) centroids differ: {gc} vs {oc}"
        exact += int(np.sum(gc == oc))
        total += k
        if err is not None:
            np.testing.assert_allclose(float(err[i]), ora["err"][i, bi], rtol=ERR_RTOL, atol=1e-30, err_msg=f"{label} row {i}")
        if codes is not None:
            want = ora["codes"][bi, i]
            d = np.nonzero(codes[i] != want)[0]
            assert len(d) <= (1.0 - LABEL_AGREE) * len(want) + 1, f"{label}: row {i}: {len(d)} labels differ"
            for j in d:
                lo, hi = sorted((int(codes[i, j]), int(want[j])))
                assert hi == lo + 1, f"{label}: labels differ by more than one cluster"
                x = x_values[i, j]
                assert any(abs(x - 0.5 * (c[lo] + c[hi])) <= 4 * np.spacing(np.float32(abs(0.5 * (c[lo] + c[hi]))))
                           for c in (gc, oc)), f"{label}: label mismatch away from a midpoint (row {i}, col {j})"
    return exact / max(total, 1)


def unpack_row(words, cols, b):
    bits = np.unpackbits(np.ascontiguousarray(words).view(np.uint8), bitorder="little")[:cols * b].reshape(cols, b)
    return (bits * (1 << np.arange(b))).sum(axis=1).astype(np.uint8)
