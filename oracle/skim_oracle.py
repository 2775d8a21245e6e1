"""ctypes binding of the CPU oracle (``skim_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, the smoke check and the
benchmark's CPU-baseline leg.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "skim_oracle.c")
_LIB = os.path.join(_HERE, "libskim_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over rows only); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-fPIC",
               "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.skim_oracle_row_stride_words.restype = C.c_int64
        _lib.skim_oracle_row_stride_words.argtypes = [C.c_int64, C.c_int]
        _lib.skim_oracle_float_to_half.restype = C.c_uint16
        _lib.skim_oracle_float_to_half.argtypes = [C.c_float]
        _lib.skim_oracle_half_to_float.restype = C.c_float
        _lib.skim_oracle_half_to_float.argtypes = [C.c_uint16]
    return _lib


def num_threads() -> int:
    return int(lib().skim_oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _bit_array(bit_set):
    arr = np.ascontiguousarray(bit_set, dtype=np.int32)
    return arr, int(sum(1 << int(b) for b in arr))


def kmeans_row(x, g, k, iters, round_fp32=True, want_trace=False):
    """One row: returns dict(c, label, err, trace, n_distinct)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    m = x.shape[0]
    c = np.zeros(k, dtype=np.float64)
    label = np.zeros(m, dtype=np.int32)
    err = C.c_double(0.0)
    nd = C.c_int(0)
    trace = np.zeros(2 * iters + 1, dtype=np.float64) if want_trace else None
    rc = lib().skim_oracle_kmeans_row(_p(x), _p(g), C.c_int64(m), C.c_int(k), C.c_int(iters),
                                      C.c_int(1 if round_fp32 else 0), _p(c), _p(label),
                                      C.byref(err), _p(trace), C.byref(nd))
    if rc:
        raise ValueError(f"skim_oracle_kmeans_row failed ({rc})")
    return dict(c=c, label=label, err=err.value, trace=trace, n_distinct=nd.value)


def cluster_rows(W, importance, bit_set, iters, s=None, row_bits=None, round_fp32=True,
                 want_codes=True, want_trace=False):
    """All rows at all bit-widths.  ``W`` float16 [rows, cols]; ``importance`` float32.

    Returns dict(centroids float64 [rows, sum 2^b], codes uint8 [n_bits, rows, cols] or None,
    err float64 [rows, n_bits], trace or None).
    """
    W = np.ascontiguousarray(W)
    assert W.dtype == np.float16 and W.ndim == 2
    importance = np.ascontiguousarray(importance, dtype=np.float32)
    assert importance.shape == W.shape
    rows, cols = W.shape
    bits, sumk = _bit_array(bit_set)
    nb = len(bits)
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
        assert s.shape == (cols,)
    if row_bits is not None:
        row_bits = np.ascontiguousarray(row_bits, dtype=np.uint8)
    centroids = np.zeros((rows, sumk), dtype=np.float64)
    codes = np.zeros((nb, rows, cols), dtype=np.uint8) if want_codes else None
    err = np.zeros((rows, nb), dtype=np.float64)
    trace = np.zeros((rows, nb, 2 * iters + 1), dtype=np.float64) if want_trace else None
    rc = lib().skim_oracle_cluster_rows(_p(W.view(np.uint16)), _p(importance), C.c_int64(rows),
                                        C.c_int64(cols), C.c_int64(cols), _p(s), _p(row_bits),
                                        _p(bits), C.c_int(nb), C.c_int(iters),
                                        C.c_int(1 if round_fp32 else 0), _p(centroids), _p(codes),
                                        _p(err), _p(trace))
    if rc:
        raise ValueError(f"skim_oracle_cluster_rows failed ({rc})")
    return dict(centroids=centroids, codes=codes, err=err, trace=trace)


def kmeans_exact_row(x, g, ks):
    """Optimal weighted 1-D K-means of one row for every cluster count in ``ks`` (ascending): returns
    (centroids: concatenated blocks, err [len(ks)])."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    ks = np.ascontiguousarray(ks, dtype=np.int32)
    c = np.zeros(int(ks.sum()), dtype=np.float64)
    err = np.zeros(len(ks), dtype=np.float64)
    rc = lib().skim_oracle_kmeans_exact_row(_p(x), _p(g), C.c_int64(x.shape[0]), _p(ks), C.c_int(len(ks)), _p(c), _p(err))
    if rc:
        raise ValueError(f"skim_oracle_kmeans_exact_row failed ({rc})")
    return c, err


def cluster_rows_exact(W, importance, bit_set, s=None):
    """Exact (optimal) clustering of all rows at all widths: dict(centroids float64 [rows, sum 2^b], err [rows, n_bits])."""
    W = np.ascontiguousarray(W)
    assert W.dtype == np.float16 and W.ndim == 2
    importance = np.ascontiguousarray(importance, dtype=np.float32)
    rows, cols = W.shape
    bits, sumk = _bit_array(bit_set)
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
    centroids = np.zeros((rows, sumk), dtype=np.float64)
    err = np.zeros((rows, len(bits)), dtype=np.float64)
    rc = lib().skim_oracle_cluster_rows_exact(_p(W.view(np.uint16)), _p(importance), C.c_int64(rows), C.c_int64(cols),
                                              C.c_int64(cols), _p(s), _p(bits), C.c_int(len(bits)), _p(centroids), _p(err))
    if rc:
        raise ValueError(f"skim_oracle_cluster_rows_exact failed ({rc})")
    return dict(centroids=centroids, err=err)


def allocate_bits(err, b_min, budget, floor_start=False, round_up=False):
    """Greedy allocation over a float32 table [rows, n_bits]; returns (bits uint8 [rows], total).
    floor_start: every row starts at floor(budget) instead of b_min.  round_up: Algorithm 1's literal
    stopping rule (until the total reaches rows * budget), i.e. the total rounded up."""
    err = np.ascontiguousarray(err, dtype=np.float32)
    rows, nb = err.shape
    bits = np.zeros(rows, dtype=np.uint8)
    total = C.c_int64(0)
    fn = lib().skim_oracle_allocate_bits_floor if floor_start else lib().skim_oracle_allocate_bits
    if round_up:
        assert not floor_start
        fn = lib().skim_oracle_allocate_bits_until
    rc = fn(_p(err), C.c_int64(rows), C.c_int(nb), C.c_int(b_min), C.c_double(budget), _p(bits), C.byref(total))
    if rc == -2:
        raise ValueError("budget outside [b_min, b_max]")
    if rc:
        raise ValueError(f"skim_oracle_allocate_bits failed ({rc})")
    return bits, total.value


def allocate_optimal(err, b_min, budget):
    """Exact minimum-error allocation with the greedy's total (dynamic programme); returns (bits, total, cost)."""
    err = np.ascontiguousarray(err, dtype=np.float32)
    rows, nb = err.shape
    bits = np.zeros(rows, dtype=np.uint8)
    total = C.c_int64(0)
    cost = C.c_double(0.0)
    rc = lib().skim_oracle_allocate_optimal(_p(err), C.c_int64(rows), C.c_int(nb), C.c_int(b_min), C.c_double(budget),
                                            _p(bits), C.byref(total), C.byref(cost))
    if rc == -2:
        raise ValueError("budget outside [b_min, b_max]")
    if rc:
        raise ValueError(f"skim_oracle_allocate_optimal failed ({rc})")
    return bits, total.value, cost.value


def row_stride_words(cols, b):
    return int(lib().skim_oracle_row_stride_words(C.c_int64(cols), C.c_int(b)))


def emit(W, bits, centroids, bit_set, s=None):
    """Packed codes, row order, group starts/offsets, fp16 LUT and unpacked codes."""
    W = np.ascontiguousarray(W)
    assert W.dtype == np.float16
    rows, cols = W.shape
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    centroids = np.ascontiguousarray(centroids, dtype=np.float32)
    bs, sumk = _bit_array(bit_set)
    nb = len(bs)
    assert centroids.shape == (rows, sumk)
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
    kmax = 1 << int(bs[-1])
    max_words = rows * row_stride_words(cols, int(bs[-1]))
    packed = np.zeros(max_words, dtype=np.uint32)
    row_order = np.zeros(rows, dtype=np.int32)
    group_start = np.zeros(nb + 1, dtype=np.int64)
    group_word = np.zeros(nb + 1, dtype=np.int64)
    lut = np.zeros((rows, kmax), dtype=np.uint16)
    codes = np.zeros((rows, cols), dtype=np.uint8)
    rc = lib().skim_oracle_emit(_p(W.view(np.uint16)), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols),
                                _p(s), _p(bits), _p(centroids), _p(bs), C.c_int(nb), _p(packed),
                                _p(row_order), _p(group_start), _p(group_word), _p(lut), _p(codes))
    if rc:
        raise ValueError(f"skim_oracle_emit failed ({rc})")
    return dict(packed=packed[:int(group_word[-1])], row_order=row_order, group_start=group_start,
                group_word=group_word, lut=lut, codes=codes)


def _packed_args(em, bit_set):
    bs, _ = _bit_array(bit_set)
    packed = np.ascontiguousarray(em["packed"], dtype=np.uint32)
    if packed.size == 0:
        packed = np.zeros(4, dtype=np.uint32)
    return (bs, packed, np.ascontiguousarray(em["row_order"], dtype=np.int32),
            np.ascontiguousarray(em["group_start"], dtype=np.int64), np.ascontiguousarray(em["group_word"], dtype=np.int64),
            np.ascontiguousarray(em["lut"], dtype=np.uint16))


def dequantize(em, cols, bit_set, s=None):
    """Dequantised weights (float16 [rows, cols]) from an emit() result."""
    bs, packed, row_order, gs, gw, lut = _packed_args(em, bit_set)
    rows = lut.shape[0]
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
    out = np.zeros((rows, cols), dtype=np.uint16)
    rc = lib().skim_oracle_dequantize(_p(packed), _p(row_order), _p(gs), _p(gw), _p(lut), _p(s), C.c_int64(rows),
                                      C.c_int64(cols), _p(bs), C.c_int(len(bs)), _p(out))
    if rc:
        raise ValueError(f"skim_oracle_dequantize failed ({rc})")
    return out.view(np.float16)


def matvec(em, cols, bit_set, x, s=None):
    """y = Wq x from the packed form; returns (y float64 [rows], sum of |terms| float64 [rows])."""
    bs, packed, row_order, gs, gw, lut = _packed_args(em, bit_set)
    rows = lut.shape[0]
    x = np.ascontiguousarray(x)
    assert x.dtype == np.float16 and x.shape == (cols,)
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
    y = np.zeros(rows, dtype=np.float64)
    mag = np.zeros(rows, dtype=np.float64)
    rc = lib().skim_oracle_matvec(_p(packed), _p(row_order), _p(gs), _p(gw), _p(lut), _p(s), _p(x.view(np.uint16)),
                                  C.c_int64(rows), C.c_int64(cols), _p(bs), C.c_int(len(bs)), _p(y), _p(mag))
    if rc:
        raise ValueError(f"skim_oracle_matvec failed ({rc})")
    return y, mag


def residual(W, centroids, bit_set, width=None, row_bits=None, s=None, exp2=8):
    """Scaled residual float16 [rows, cols]: binary16((float(w) - c[label] * alpha) * 2^exp2); the operand of err_lfull."""
    W = np.ascontiguousarray(W)
    assert W.dtype == np.float16
    rows, cols = W.shape
    centroids = np.ascontiguousarray(centroids, dtype=np.float32)
    bs, sumk = _bit_array(bit_set)
    assert centroids.shape == (rows, sumk)
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
    if row_bits is not None:
        row_bits = np.ascontiguousarray(row_bits, dtype=np.uint8)
    D = np.zeros((rows, cols), dtype=np.uint16)
    rc = lib().skim_oracle_residual(_p(W.view(np.uint16)), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols), _p(s),
                                    _p(row_bits), C.c_int(0 if width is None else int(width)), _p(centroids), _p(bs),
                                    C.c_int(len(bs)), C.c_int(exp2), _p(D), C.c_int64(cols))
    if rc:
        raise ValueError(f"skim_oracle_residual failed ({rc})")
    return D.view(np.float16)


def err_lfull(D, H, exp2=8):
    """L-full error d H d^T / 4^exp2 of every row of D (float16) for H (float16 [cols, cols]); returns (err, mag)."""
    D = np.ascontiguousarray(D)
    H = np.ascontiguousarray(H)
    assert D.dtype == np.float16 and H.dtype == np.float16
    rows, cols = D.shape
    assert H.shape == (cols, cols)
    err = np.zeros(rows, dtype=np.float64)
    mag = np.zeros(rows, dtype=np.float64)
    rc = lib().skim_oracle_err_lfull(_p(D.view(np.uint16)), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols),
                                     _p(H.view(np.uint16)), C.c_int64(cols), C.c_int(exp2), _p(err), _p(mag))
    if rc:
        raise ValueError(f"skim_oracle_err_lfull failed ({rc})")
    return err, mag


def scale_loss_grad(W, importance, labels, alpha, want_grad=True):
    W = np.ascontiguousarray(W)
    assert W.dtype == np.float16
    importance = np.ascontiguousarray(importance, dtype=np.float32)
    labels = np.ascontiguousarray(labels, dtype=np.uint8)
    alpha = np.ascontiguousarray(alpha, dtype=np.float64)
    rows, cols = W.shape
    loss = C.c_double(0.0)
    grad = np.zeros(cols, dtype=np.float64) if want_grad else None
    rc = lib().skim_oracle_scale_loss_grad(_p(W.view(np.uint16)), _p(importance), C.c_int64(rows),
                                           C.c_int64(cols), C.c_int64(cols), _p(labels), _p(alpha),
                                           C.byref(loss), _p(grad))
    if rc:
        raise ValueError(f"skim_oracle_scale_loss_grad failed ({rc})")
    return loss.value, grad


def scale_loss_grad_lfull(W, importance, labels, alpha, H, exp2=8, round_d=True, want_grad=True):
    """L-full loss sum_i d_i H d_i^T of the scaling vector and its gradient (labels fixed)."""
    W = np.ascontiguousarray(W)
    H = np.ascontiguousarray(H)
    assert W.dtype == np.float16 and H.dtype == np.float16
    importance = np.ascontiguousarray(importance, dtype=np.float32)
    labels = np.ascontiguousarray(labels, dtype=np.uint8)
    alpha = np.ascontiguousarray(alpha, dtype=np.float64)
    rows, cols = W.shape
    loss = C.c_double(0.0)
    grad = np.zeros(cols, dtype=np.float64) if want_grad else None
    rc = lib().skim_oracle_scale_loss_grad_lfull(_p(W.view(np.uint16)), _p(importance), C.c_int64(rows), C.c_int64(cols),
                                                 C.c_int64(cols), _p(labels), _p(alpha), _p(H.view(np.uint16)), C.c_int64(cols),
                                                 C.c_int(exp2), C.c_int(1 if round_d else 0), C.byref(loss), _p(grad))
    if rc:
        raise ValueError(f"skim_oracle_scale_loss_grad_lfull failed ({rc})")
    return loss.value, grad


def scale_update_lfull(W, importance, labels, alpha, H, steps=120, exp2=8, round_d=True, lr0=0.01, decay=0.5,
                       decay_every=40, beta1=0.9, beta2=0.999, eps=1e-8):
    """Returns (alpha float64 [cols] after `steps` Adam steps on the L-full loss, loss trace [steps])."""
    W = np.ascontiguousarray(W)
    H = np.ascontiguousarray(H)
    assert W.dtype == np.float16 and H.dtype == np.float16
    importance = np.ascontiguousarray(importance, dtype=np.float32)
    labels = np.ascontiguousarray(labels, dtype=np.uint8)
    alpha = np.array(alpha, dtype=np.float64, copy=True)
    rows, cols = W.shape
    trace = np.zeros(steps, dtype=np.float64)
    rc = lib().skim_oracle_scale_update_lfull(_p(W.view(np.uint16)), _p(importance), C.c_int64(rows), C.c_int64(cols),
                                              C.c_int64(cols), _p(labels), _p(H.view(np.uint16)), C.c_int64(cols),
                                              C.c_int(exp2), C.c_int(1 if round_d else 0), _p(alpha), C.c_int(steps),
                                              C.c_double(lr0), C.c_double(decay), C.c_int(decay_every), C.c_double(beta1),
                                              C.c_double(beta2), C.c_double(eps), _p(trace))
    if rc:
        raise ValueError(f"skim_oracle_scale_update_lfull failed ({rc})")
    return alpha, trace


def scale_update(W, importance, labels, alpha, steps=120, lr0=0.01, decay=0.5, decay_every=40,
                 beta1=0.9, beta2=0.999, eps=1e-8):
    """Returns (alpha float64 [cols] after `steps` Adam steps, loss trace [steps])."""
    W = np.ascontiguousarray(W)
    assert W.dtype == np.float16
    importance = np.ascontiguousarray(importance, dtype=np.float32)
    labels = np.ascontiguousarray(labels, dtype=np.uint8)
    alpha = np.array(alpha, dtype=np.float64, copy=True)
    rows, cols = W.shape
    trace = np.zeros(steps, dtype=np.float64)
    rc = lib().skim_oracle_scale_update(_p(W.view(np.uint16)), _p(importance), C.c_int64(rows),
                                        C.c_int64(cols), C.c_int64(cols), _p(labels), _p(alpha),
                                        C.c_int(steps), C.c_double(lr0), C.c_double(decay),
                                        C.c_int(decay_every), C.c_double(beta1), C.c_double(beta2),
                                        C.c_double(eps), _p(trace))
    if rc:
        raise ValueError(f"skim_oracle_scale_update failed ({rc})")
    return alpha, trace
