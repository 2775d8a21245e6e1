"""Seeded synthetic inputs: weight matrices, importance tables, scale vectors, error tables.

This module holds no arithmetic of the quantisation method itself; it only draws
random numbers.  Both the CPU oracle's tests and the CUDA path's tests/benchmarks
take their inputs from here, so the two are always fed identical bytes.

Recipe (stands in for LLaMA weights and squared calibration gradients, which are
not available offline).  A matrix is generated in blocks of ``BLOCK_ROWS`` rows;
block ``k`` of a matrix with seed ``s`` uses ``numpy.random.Generator(PCG64(
SeedSequence([s, k])))`` and draws, in this fixed order, for its ``r x cols``
elements:

1. ``v = standard_normal(float32) * sigma_w``                (sigma_w = 0.02)
2. ``mask = random(float32) < outlier_frac``                 (outlier_frac = 1e-3)
3. ``v[mask] = 0.2 * standard_t(df=3, size=mask.sum())``      (heavy-tailed outliers)
4. ``W = v.astype(float16)``                                  (round to nearest even)
5. ``importance = exp(importance_sigma * standard_normal(float32)).astype(float32)``

Because every block has its own stream, any row range can be generated without
generating the rest of the matrix.
"""
from __future__ import annotations

import numpy as np

BLOCK_ROWS = 256

# LLaMA linear-layer shapes (rows = output channels).
LLAMA7B_ATTN = (4096, 4096)
LLAMA7B_GATE_UP = (11008, 4096)
LLAMA7B_DOWN = (4096, 11008)
LLAMA65B_GATE_UP = (22016, 8192)
LLAMA65B_DOWN = (8192, 22016)

# One LLaMA-7B transformer block: 4 attention projections, gate, up, down.
LLAMA7B_BLOCK = [LLAMA7B_ATTN] * 4 + [LLAMA7B_GATE_UP] * 2 + [LLAMA7B_DOWN]


def _block(rows, cols, seed, k, sigma_w, outlier_frac, importance_sigma):
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(k)])))
    n = rows * cols
    v = rng.standard_normal(n, dtype=np.float32) * np.float32(sigma_w)
    if outlier_frac > 0.0:
        mask = rng.random(n, dtype=np.float32) < np.float32(outlier_frac)
        cnt = int(mask.sum())
        if cnt:
            v[mask] = (0.2 * rng.standard_t(3.0, size=cnt)).astype(np.float32)
    w = v.astype(np.float16).reshape(rows, cols)
    z = rng.standard_normal(n, dtype=np.float32)
    g = np.exp(np.float32(importance_sigma) * z).astype(np.float32).reshape(rows, cols)
    return w, g


def make_rows(rows, cols, seed, row_start=0, row_count=None, *, sigma_w=0.02,
              outlier_frac=1e-3, importance_sigma=1.5):
    """Rows ``[row_start, row_start+row_count)`` of the ``rows x cols`` matrix with this seed.

    Returns ``(W float16 [row_count, cols], importance float32 [row_count, cols])``.
    """
    if row_count is None:
        row_count = rows - row_start
    if row_start < 0 or row_count < 0 or row_start + row_count > rows:
        raise ValueError("row range outside the matrix")
    w_out = np.empty((row_count, cols), dtype=np.float16)
    g_out = np.empty((row_count, cols), dtype=np.float32)
    r = row_start
    end = row_start + row_count
    while r < end:
        k = r // BLOCK_ROWS
        b0 = k * BLOCK_ROWS
        b_rows = min(BLOCK_ROWS, rows - b0)
        w, g = _block(b_rows, cols, seed, k, sigma_w, outlier_frac, importance_sigma)
        lo = r - b0
        hi = min(end, b0 + b_rows) - b0
        w_out[r - row_start:r - row_start + (hi - lo)] = w[lo:hi]
        g_out[r - row_start:r - row_start + (hi - lo)] = g[lo:hi]
        r = b0 + hi
    return w_out, g_out


def make_matrix(rows, cols, seed, **kw):
    """The whole ``rows x cols`` matrix: ``(W float16, importance float32)``."""
    return make_rows(rows, cols, seed, 0, rows, **kw)


def make_scale(cols, seed, spread=0.25):
    """A positive column scale vector ``s`` (float32 [cols]), log-normal around 1."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), 0x5CA1E])))
    return np.exp(np.float32(spread) * rng.standard_normal(cols, dtype=np.float32)).astype(np.float32)


def make_gram(cols, seed, samples=64, *, correlated=0.3, outlier_channels=4):
    """A synthetic layer-input Gram matrix H = X X^T / samples (float16 [cols, cols], symmetric) from
    ``samples`` random input vectors: independent N(0,1) channels plus a shared component of weight
    ``correlated`` (so off-diagonal entries are not negligible) and a few channels of 8x magnitude, as
    LLM activations have.  Stands in for calibration activations, which are not available offline."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), 0x6A2])))
    X = rng.standard_normal((cols, samples), dtype=np.float32)
    X += np.float32(correlated) * rng.standard_normal((1, samples), dtype=np.float32)
    if outlier_channels:
        X[rng.choice(cols, size=min(outlier_channels, cols), replace=False)] *= np.float32(8.0)
    H = (X.astype(np.float64) @ X.astype(np.float64).T) / samples
    H16 = H.astype(np.float16)
    return np.ascontiguousarray(np.triu(H16) + np.triu(H16, 1).T)


def make_error_table(rows, n_bits, seed, *, monotone=True, ties=False):
    """A synthetic error table (float32 [rows, n_bits]) for allocator tests.

    ``monotone`` gives every row non-increasing marginal gains (a convex, decreasing
    error curve); otherwise rows are arbitrary positive numbers (gains may be negative
    or increase with the bit-width).  ``ties`` quantises values coarsely so that many
    gains are exactly equal.
    """
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), 0xE77])))
    if monotone:
        gains = np.sort(rng.lognormal(0.0, 1.5, size=(rows, n_bits - 1)), axis=1)[:, ::-1]
        if ties:
            gains = np.ceil(gains * 2.0) / 2.0
        tail = rng.lognormal(-2.0, 0.5, size=(rows, 1))
        if ties:
            tail = np.ceil(tail * 2.0) / 2.0
        err = np.concatenate([gains, tail], axis=1)[:, ::-1].cumsum(axis=1)[:, ::-1]
    else:
        err = rng.lognormal(0.0, 1.0, size=(rows, n_bits))
        if ties:
            err = np.ceil(err * 2.0) / 2.0
    return np.ascontiguousarray(err, dtype=np.float32)


# The five benchmark configurations.  ``matrices`` lists (rows, cols, seed).
def config(idx):
    """Workload description for configuration ``idx`` (1..5)."""
    if idx == 1:
        return dict(matrices=[(256, 512, 0)], outlier_frac=0.0, importance_sigma=1.0,
                    bit_set=[1, 2, 3, 4], iters=30, budgets=[3.2], scale_rounds=0)
    if idx == 2:
        return dict(matrices=[LLAMA7B_ATTN + (2000,)], outlier_frac=1e-3, importance_sigma=1.5,
                    bit_set=[1, 2, 3, 4], iters=50, budgets=[3.0], scale_rounds=0)
    if idx == 3:
        return dict(matrices=[LLAMA7B_GATE_UP + (3000,), LLAMA7B_DOWN + (3001,)], outlier_frac=1e-3,
                    importance_sigma=1.5, bit_set=[1, 2, 3, 4], iters=50, budgets=[2.5, 3.0],
                    scale_rounds=0)
    if idx == 4:
        mats = []
        for blk in range(32):
            for j, shp in enumerate(LLAMA7B_BLOCK):
                mats.append(shp + (4000 + blk * len(LLAMA7B_BLOCK) + j,))
        return dict(matrices=mats, outlier_frac=1e-3, importance_sigma=1.5, bit_set=[1, 2, 3, 4],
                    iters=50, budgets=[2.25, 2.5, 3.0], scale_rounds=0)
    if idx == 5:
        return dict(matrices=[LLAMA65B_GATE_UP + (5000,), LLAMA65B_DOWN + (5001,)], outlier_frac=1e-3,
                    importance_sigma=2.0, bit_set=[1, 2, 3, 4], iters=50, budgets=[3.0],
                    scale_rounds=5)
    raise ValueError("config index must be 1..5")
