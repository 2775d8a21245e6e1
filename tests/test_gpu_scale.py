"""GPU parity: the scaling-vector update (Algorithm 2, inner repeat) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs

pytestmark = pytest.mark.gpu
BITS = [1, 2, 3, 4]


def _labels(oracle, w, g, bits):
    res = oracle.cluster_rows(w, g, BITS, 15, row_bits=bits)
    rows = w.shape[0]
    return np.stack([res["codes"][int(b) - 1, i] for i, b in enumerate(bits)]).astype(np.uint8)


@pytest.mark.parametrize("rows,cols,steps", [(16, 64, 1), (40, 520, 7), (300, 257, 45), (700, 1024, 120)])
def test_scale_update_matches_oracle(ctx, oracle, rows, cols, steps):
    w, g = inputs.make_rows(rows, cols, 50 + rows, outlier_frac=0.01)
    bits = (np.arange(rows) % 4 + 1).astype(np.uint8)
    labels = _labels(oracle, w, g, bits)
    a0 = inputs.make_scale(cols, 3, spread=0.05)
    want, trace = oracle.scale_update(w, g, labels, a0.astype(np.float64), steps=steps)
    ctx.reserve(rows, cols)
    alpha = torch.from_numpy(a0.copy()).cuda()
    got_trace = ctx.scale_update(torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(),
                                 torch.from_numpy(labels).cuda(), alpha, steps=steps)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    # both sides carry alpha in binary64 and differ only in summation order (Adam's normalised
    # step amplifies that where a gradient entry is near zero); the result is returned as binary32
    np.testing.assert_allclose(got_trace.cpu().numpy(), trace, rtol=1e-7)
    np.testing.assert_allclose(alpha.cpu().numpy().astype(np.float64), want, rtol=1e-6, atol=0)


def test_scale_update_wide_rows(ctx, oracle):
    rows, cols = 6, 22016
    w, g = inputs.make_rows(8192, cols, 5001, 0, rows, importance_sigma=2.0)
    bits = np.array([1, 2, 3, 4, 4, 3], np.uint8)
    labels = _labels(oracle, w, g, bits)
    a0 = np.ones(cols, np.float32)
    want, trace = oracle.scale_update(w, g, labels, a0.astype(np.float64), steps=5)
    ctx.reserve(rows, cols)
    alpha = torch.from_numpy(a0.copy()).cuda()
    got = ctx.scale_update(torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(), torch.from_numpy(labels).cuda(),
                           alpha, steps=5)
    np.testing.assert_allclose(got.cpu().numpy(), trace, rtol=1e-7)
    np.testing.assert_allclose(alpha.cpu().numpy().astype(np.float64), want, rtol=1e-6)
