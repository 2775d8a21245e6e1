"""GPU parity of skim_cluster_rows_exact (the optimum of the clustering objective per row) against the oracle's
plain dynamic programme.  The optimum VALUE is unique and is compared; the partition is not unique at ties, so
the centroids are compared where both sides chose the same partition and are otherwise checked for validity:
ascending, and realising the optimum under the nearest-centroid assignment (numpy)."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs
from test_gpu_cluster import _degenerate_rows, _values

pytestmark = pytest.mark.gpu
BITS = [1, 2, 3, 4]


def _check(ctx, oracle, w, g, bit_set, s=None, label=""):
    rows, cols = w.shape
    ctx.reserve(rows, cols)
    ctx.apply_scale(torch.from_numpy(s).cuda() if s is not None else None)
    cent, err = ctx.cluster_rows_exact(torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(), bit_set)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    ctx.apply_scale(None)
    cent, err = cent.cpu().numpy().astype(np.float64), err.cpu().numpy().astype(np.float64)
    ora = oracle.cluster_rows_exact(w, g, bit_set, s=s)
    x = _values(w, s)
    scale = (g.astype(np.float64) * x * x).sum(axis=1)
    # the optimum itself (binary32 output of a binary64 computation)
    np.testing.assert_allclose(err, ora["err"], rtol=1e-6, atol=1e-12 * scale.max(), err_msg=label)
    off, same = 0, 0
    for bi, b in enumerate(bit_set):
        k = 1 << b
        c = cent[:, off:off + k]
        assert np.all(np.diff(c, axis=1) >= 0), label
        oc = ora["centroids"][:, off:off + k]
        close = np.all(np.abs(c - oc) <= 1e-6 * np.maximum(np.abs(oc), 1e-3 * np.abs(oc).max(axis=1, keepdims=True)), axis=1)
        same += int(close.sum())
        for i in range(rows):
            lab = np.argmin(np.abs(x[i][:, None] - c[i][None, :]), axis=1)
            realised = np.sum(g[i].astype(np.float64) * (x[i] - c[i][lab]) ** 2)
            assert realised <= ora["err"][i, bi] * (1 + 1e-5) + 1e-12 * scale[i], f"{label}: row {i} width {b}"
            assert realised >= ora["err"][i, bi] * (1 - 1e-6) - 1e-12 * scale[i], f"{label}: row {i} width {b}"
        off += k
    return same / (rows * len(bit_set)), err


@pytest.mark.parametrize("cols", [1, 2, 15, 17, 33, 100, 513, 1000, 2049])
def test_exact_ragged_column_counts(ctx, oracle, cols):
    w, g = inputs.make_rows(7, cols, 900 + cols)
    same, _ = _check(ctx, oracle, w, g, BITS, label=f"cols={cols}")
    assert same > 0.9


@pytest.mark.parametrize("cols", [64, 600])
def test_exact_degenerate_rows(ctx, oracle, cols):
    w, g = _degenerate_rows(cols)
    _, err = _check(ctx, oracle, w, g, BITS, label="degenerate")
    assert np.all(err[0] == 0) and np.all(err[1] == 0) and np.all(err[7] == 0)
    assert np.all(err[2, 1:] == 0) and np.all(err[4, 3:] == 0)


@pytest.mark.parametrize("bit_set", [[1], [4], [2, 3], [1, 2, 3]])
def test_exact_other_bit_sets_and_scale(ctx, oracle, bit_set):
    w, g = inputs.make_rows(8, 777, 37)
    _check(ctx, oracle, w, g, bit_set, label=str(bit_set))
    _check(ctx, oracle, w, g, bit_set, s=inputs.make_scale(777, 5), label=f"scaled {bit_set}")


@pytest.mark.parametrize("cols,seed,nrows", [(4096, 2000, 12), (11008, 3001, 6)])
def test_exact_llama_row_lengths_and_gain_over_lloyd(ctx, oracle, cols, seed, nrows):
    w, g = inputs.make_rows(4096, cols, seed, 256, nrows)
    same, err = _check(ctx, oracle, w, g, BITS, label=f"cols={cols}")
    assert same > 0.9
    _, _, lloyd = ctx.cluster_rows(torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(), BITS, 50)
    lloyd = lloyd.cpu().numpy().astype(np.float64)
    assert np.all(err <= lloyd * (1 + 1e-6))     # 50 iterations from the quantile start never beat the optimum
    assert np.all(err[:, 0] >= 0.9 * lloyd[:, 0])   # and with two centroids they all but reach it


def test_exact_argument_errors(ctx, skimlib):
    w, g = inputs.make_rows(4, 256, 5)
    W, G = torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda()
    ctx.reserve(4, 256)
    with pytest.raises(skimlib.SkimError) as e:
        ctx.cluster_rows_exact(W, G, BITS, scratch=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -5
    with pytest.raises(skimlib.SkimError) as e:
        ctx.cluster_rows_exact(W, G, [1, 3])
    assert e.value.code == -3
