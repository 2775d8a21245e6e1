"""GPU parity: skim_cluster_rows / skim_cluster_rows_at against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs
from parity import check_cluster

pytestmark = pytest.mark.gpu
BITS = [1, 2, 3, 4]


def _gpu_cluster(ctx, w, g, bit_set, iters, s=None, codes=True):
    W = torch.from_numpy(w).cuda()
    G = torch.from_numpy(g).cuda()
    ctx.reserve(w.shape[0], w.shape[1])
    if s is not None:
        ctx.apply_scale(torch.from_numpy(s).cuda())
    else:
        ctx.apply_scale(None)
    cent, cd, err = ctx.cluster_rows(W, G, bit_set, iters, want_codes=codes)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    return cent.cpu().numpy(), err.cpu().numpy(), (cd.cpu().numpy() if codes else None)


def _values(w, s):
    x = w.astype(np.float32)
    if s is not None:
        x = x * (np.float32(1.0) / s)
    return x.astype(np.float64)


def test_config1_full(ctx, oracle):
    cfg = inputs.config(1)
    rows, cols, seed = cfg["matrices"][0]
    w, g = inputs.make_matrix(rows, cols, seed, outlier_frac=cfg["outlier_frac"], importance_sigma=cfg["importance_sigma"])
    ora = oracle.cluster_rows(w, g, BITS, cfg["iters"])
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, cfg["iters"])
    exact = check_cluster(ora, cent, err, codes, _values(w, None), BITS, label="config1")
    assert exact > 0.99      # fp32 centroids agree bit for bit almost everywhere


@pytest.mark.parametrize("cols", [1, 2, 15, 16, 17, 33, 100, 511, 513, 1000, 2049, 4097, 5000])
def test_ragged_column_counts(ctx, oracle, cols):
    w, g = inputs.make_rows(9, cols, 700 + cols)
    ora = oracle.cluster_rows(w, g, BITS, 12)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 12)
    check_cluster(ora, cent, err, codes, _values(w, None), BITS, label=f"cols={cols}")


@pytest.mark.parametrize("iters", [0, 1, 2, 50, 200])
def test_iteration_counts(ctx, oracle, iters):
    w, g = inputs.make_rows(16, 1536, 31)
    ora = oracle.cluster_rows(w, g, BITS, iters)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, iters)
    check_cluster(ora, cent, err, codes, _values(w, None), BITS, label=f"iters={iters}")


@pytest.mark.parametrize("bit_set", [[1], [4], [2, 3], [3, 4], [1, 2, 3]])
def test_other_bit_sets(ctx, oracle, bit_set):
    w, g = inputs.make_rows(12, 777, 37)
    ora = oracle.cluster_rows(w, g, bit_set, 20)
    cent, err, codes = _gpu_cluster(ctx, w, g, bit_set, 20)
    check_cluster(ora, cent, err, codes, _values(w, None), bit_set, label=str(bit_set))


def _degenerate_rows(cols):
    w, g = inputs.make_rows(12, cols, 55)
    w[0, :] = np.float16(0.25)                                  # one distinct value
    w[1, :] = np.where(np.arange(cols) % 2 == 0, np.float16(-1.0), np.float16(1.0))   # two
    w[2, :] = (np.arange(cols) % 3).astype(np.float16)          # three
    w[3, :] = (np.arange(cols) % 5).astype(np.float16) - 2      # five
    w[4, :] = (np.arange(cols) % 16).astype(np.float16) / 8     # sixteen
    w[5, :] = (np.arange(cols) % 17).astype(np.float16) / 8     # seventeen
    w[6, : cols // 2] = 0.0                                     # half zeros: duplicate init centroids
    w[7, :] = np.where(np.arange(cols) % 2 == 0, np.float16(0.0), np.float16(-0.0))   # +0 and -0 are one value
    w[8, : (cols * 9) // 10] = np.float16(0.0123)               # a heavy clump
    w[9, :] = np.round(w[9, :].astype(np.float32) * 32).astype(np.float16) / np.float16(32)  # coarse grid
    g[10, :] = 0.0                                              # no importance at all
    g[11, ::2] = 0.0                                            # half the elements weightless
    return w, g


@pytest.mark.parametrize("cols", [64, 1000])
def test_degenerate_rows(ctx, oracle, cols):
    w, g = _degenerate_rows(cols)
    ora = oracle.cluster_rows(w, g, BITS, 15)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 15)
    check_cluster(ora, cent, err, codes, _values(w, None), BITS, label="degenerate")
    assert np.all(err[0] == 0) and np.all(err[1] == 0) and np.all(err[7] == 0)
    assert np.all(err[2, 1:] == 0) and np.all(err[4, 3:] == 0)


@pytest.mark.parametrize("cols", [33, 512, 3000])
def test_scaled_rows(ctx, oracle, cols):
    w, g = inputs.make_rows(10, cols, 91)
    s = inputs.make_scale(cols, 17)
    ora = oracle.cluster_rows(w, g, BITS, 20, s=s)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 20, s=s)
    check_cluster(ora, cent, err, codes, _values(w, s), BITS, label="scaled")
    # removing the scale brings back the unscaled result
    ora0 = oracle.cluster_rows(w, g, BITS, 20)
    cent0, err0, codes0 = _gpu_cluster(ctx, w, g, BITS, 20)
    check_cluster(ora0, cent0, err0, codes0, _values(w, None), BITS, label="unscaled again")


def test_scaled_degenerate_rows(ctx, oracle):
    w, g = _degenerate_rows(300)
    s = np.full(300, 0.5, np.float32)
    ora = oracle.cluster_rows(w, g, BITS, 10, s=s)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 10, s=s)
    check_cluster(ora, cent, err, codes, _values(w, s), BITS, label="scaled degenerate")


@pytest.mark.parametrize("cols,seed,sigma", [(4096, 2000, 1.5), (11008, 3001, 1.5), (8192, 5000, 2.0), (22016, 5001, 2.0)])
def test_llama_row_lengths_on_a_row_subset(ctx, oracle, cols, seed, sigma):
    """Rows are independent, so a row subset of the big matrices is compared in full."""
    rows_total = {4096: 4096, 11008: 4096, 8192: 22016, 22016: 8192}[cols]
    nrows = 48 if cols <= 11008 else 24
    w, g = inputs.make_rows(rows_total, cols, seed, 512, nrows, importance_sigma=sigma)
    ora = oracle.cluster_rows(w, g, BITS, 50)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 50)
    exact = check_cluster(ora, cent, err, codes, _values(w, None), BITS, label=f"cols={cols}")
    assert exact > 0.98


def test_scaled_long_rows(ctx, oracle):
    cols = 22016
    w, g = inputs.make_rows(8192, cols, 5001, 0, 12, importance_sigma=2.0)
    s = inputs.make_scale(cols, 3)
    ora = oracle.cluster_rows(w, g, BITS, 50, s=s)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 50, s=s)
    check_cluster(ora, cent, err, codes, _values(w, s), BITS, label="scaled 22016")


@pytest.mark.parametrize("cols", [8192, 11008, 16384])
def test_scaled_rows_at_llama_lengths(ctx, oracle, cols):
    """Scaled rows go through the 32-bit-key sort kernel; these three lengths take its three largest
    variants below the 22 016-column one (8192 is the row length of the 22016 x 8192 matrix that
    the scaling alternation runs on)."""
    w, g = inputs.make_rows(24, cols, 8100 + cols, importance_sigma=2.0)
    s = inputs.make_scale(cols, 29)
    ora = oracle.cluster_rows(w, g, BITS, 50, s=s)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 50, s=s)
    exact = check_cluster(ora, cent, err, codes, _values(w, s), BITS, label=f"scaled cols={cols}")
    assert exact > 0.98


@pytest.mark.parametrize("cols", [12296, 14000, 16384, 16392, 20000])
def test_unscaled_long_rows(ctx, oracle, cols):
    """Row lengths between the LLaMA-7B and LLaMA-65B ones (each side of the limits at which the
    fp16-key sort changes its kernel variant)."""
    w, g = inputs.make_rows(12, cols, 8200 + cols)
    ora = oracle.cluster_rows(w, g, BITS, 30)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 30)
    exact = check_cluster(ora, cent, err, codes, _values(w, None), BITS, label=f"cols={cols}")
    assert exact > 0.98


@pytest.mark.parametrize("cols,scaled", [(700, False), (11008, False), (3000, True)])
def test_contiguous_run_of_zero_importance(ctx, oracle, cols, scaled):
    """The largest 50 values of every row carry no importance at all, the rest spans many orders
    of magnitude (exp(5 N)): the top clusters of the wide widths are weightless and must keep
    their centroids, although their weight is a difference of two large rounded prefix sums."""
    rows = 16
    w, _ = inputs.make_rows(rows, cols, 8300 + cols)
    rng = np.random.default_rng(cols)
    g = np.exp(5.0 * rng.standard_normal((rows, cols))).astype(np.float32)
    s = inputs.make_scale(cols, 31) if scaled else None
    x = _values(w, s)
    top = np.argsort(x, axis=1, kind="stable")[:, -50:]
    np.put_along_axis(g, top, np.float32(0.0), axis=1)
    ora = oracle.cluster_rows(w, g, BITS, 40, s=s)
    cent, err, codes = _gpu_cluster(ctx, w, g, BITS, 40, s=s)
    check_cluster(ora, cent, err, codes, x, BITS, label="zero-importance run")


def test_cluster_rows_at_allocated_widths(ctx, oracle):
    rows, cols = 40, 1200
    w, g = inputs.make_rows(rows, cols, 123)
    bits = (np.arange(rows) * 5 % 4 + 1).astype(np.uint8)
    ora = oracle.cluster_rows(w, g, BITS, 25, row_bits=bits)
    ctx.reserve(rows, cols)
    ctx.apply_scale(None)
    cent, codes, err = ctx.cluster_rows_at(torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(),
                                           torch.from_numpy(bits).cuda(), BITS, 25)
    cent, codes, err = cent.cpu().numpy(), codes.cpu().numpy(), err.cpu().numpy()
    offs = {1: 0, 2: 2, 3: 6, 4: 14}
    for i, b in enumerate(bits):
        o, k = offs[int(b)], 1 << int(b)
        np.testing.assert_allclose(cent[i, o:o + k], ora["centroids"][i, o:o + k], rtol=1e-4)
        assert err[i] == pytest.approx(ora["err"][i, b - 1], rel=1e-5)
        assert np.mean(codes[i] == ora["codes"][b - 1, i]) >= 0.999
        # the blocks of the other widths are left alone (zero-initialised here)
        mask = np.ones(30, bool)
        mask[o:o + k] = False
        assert np.all(cent[i, mask] == 0)


def test_bad_data_sets_status_flags_and_never_faults(ctx, skimlib):
    w, g = inputs.make_rows(4, 256, 5)
    w[1, 7] = np.float16(np.nan)
    w[2, 9] = np.float16(np.inf)
    g[3, 11] = -1.0
    ctx.reserve(4, 256)
    ctx.apply_scale(None)
    ctx.cluster_rows(torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(), BITS, 5)
    assert ctx.get_status() == 3
    assert ctx.get_status() == 0          # reading clears it
    s = np.ones(256, np.float32)
    s[3] = 0.0
    ctx.apply_scale(torch.from_numpy(s).cuda())
    assert ctx.get_status() == 4
    ctx.apply_scale(None)


def test_argument_errors(ctx, skimlib):
    w, g = inputs.make_rows(4, 256, 5)
    W, G = torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda()
    with pytest.raises(skimlib.SkimError) as e:       # no workspace yet
        ctx.cluster_rows(W, G, BITS, 5)
    assert e.value.code == -5
    ctx.reserve(4, 256)
    for bad_bits in ([1, 3], [0, 1], [4, 5], [2, 1]):
        with pytest.raises(skimlib.SkimError) as e:
            ctx.cluster_rows(W, G, bad_bits, 5)
        assert e.value.code == -3
    with pytest.raises(skimlib.SkimError) as e:
        ctx.cluster_rows(W, G, BITS, -1)
    assert e.value.code == -2
    with pytest.raises(skimlib.SkimError) as e:
        ctx.cluster_rows(W, G, BITS, 5, ld=100)
    assert e.value.code == -2
    with pytest.raises(skimlib.SkimError) as e:
        ctx.cluster_rows(W, G, BITS, 5, cols=ctx.max_cols() + 1, ld=ctx.max_cols() + 1)
    assert e.value.code == -2
    ctx.apply_scale(torch.ones(128, device="cuda"))
    with pytest.raises(skimlib.SkimError) as e:       # scale length differs from cols
        ctx.cluster_rows(W, G, BITS, 5)
    assert e.value.code == -8
    ctx.apply_scale(None)
    assert ctx.max_cols() >= 22016


def test_bounds_checked_build_reports_no_violation(skimlib):
    """The checked build (every computed index into shared memory, a row record or a scratch list is
    range-checked; a violation sets a status bit and skips the access) runs the ragged column counts, the
    degenerate rows, the long rows and a scaled case, in a process of its own, with a clean status word:
    the tests it runs assert status == 0 after every clustering call."""
    import os
    import subprocess
    import sys
    from paper_2412_04180_b200 import build
    lib = build.build(checked=True)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SKIM_LIB=lib)
    cmd = [sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_cluster.py"), "-q", "-x", "-m", "gpu",
           "-k", "ragged_column_counts or degenerate_rows or unscaled_long_rows or test_scaled_rows or zero_importance",
           "-p", "no:cacheprovider"]
    res = subprocess.run(cmd, cwd=root, env=env, capture_output=True, text=True, timeout=1200)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout and "failed" not in res.stdout


def test_early_exit_switch_and_iteration_count(ctx):
    """With the converged-row shortcut off every row runs all iterations; the output is bit-identical
    (a row whose boundaries stopped moving reproduces its state), and the iteration counter says so."""
    rows, cols, iters = 40, 2048, 60
    w, g = inputs.make_rows(rows, cols, 77)
    w[3, :] = np.float16(0.5)                    # a degenerate row: no iteration changes anything
    W, G = torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda()
    ctx.reserve(rows, cols)
    ctx.apply_scale(None)
    ctx.kernel_timing(True)
    cent1, _, err1 = ctx.cluster_rows(W, G, BITS, iters)
    it_on, n_on = ctx.lloyd_iterations()
    ctx.early_exit(False)
    cent0, _, err0 = ctx.cluster_rows(W, G, BITS, iters)
    it_off, n_off = ctx.lloyd_iterations()
    ctx.early_exit(True)
    ctx.kernel_timing(False)
    torch.cuda.synchronize()
    assert torch.equal(cent0, cent1) and torch.equal(err0, err1)
    assert n_on == rows and n_off == rows
    assert it_off == rows * iters
    assert 0 < it_on <= it_off
    ctx.cluster_rows(W, G, BITS, iters)
    assert ctx.lloyd_iterations() == (0, 0)      # nothing is counted while timing is off
