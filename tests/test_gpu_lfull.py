"""GPU parity of the L-full error (Section 3.4; Section 4.2; Algorithm 3): skim_residual is bit-exact against
the oracle; skim_err_lfull (tcgen05 GEMM with the row-wise dot fused in) is within the bound its binary32
accumulation allows, (2 cols + 600) * 2^-24 * sum |d_j H_jk d_k|, and in practice two orders closer."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs

pytestmark = pytest.mark.gpu
BITS = [1, 2, 3, 4]


def _bound(cols, mag):
    return (2 * cols + 600) * 2.0 ** -24 * mag


def _check_err(ctx, oracle, D, H, exp2, rows=None, label=""):
    got = ctx.err_lfull(torch.from_numpy(D).cuda(), torch.from_numpy(H).cuda(), exp2=exp2)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    got = got.cpu().numpy().astype(np.float64)
    sel = np.arange(D.shape[0]) if rows is None else rows
    want, mag = oracle.err_lfull(D[sel], H, exp2=exp2)
    diff = np.abs(got[sel] - want)
    assert np.all(diff <= _bound(D.shape[1], mag) + 1e-30), f"{label}: {np.max(diff / np.maximum(mag, 1e-300))}"
    # what is actually observed: a few binary32 roundings relative to the magnitude sum
    assert np.all(diff <= 64 * 2.0 ** -24 * mag + 1e-30), f"{label}: {np.max(diff / np.maximum(mag, 1e-300))}"
    return got


@pytest.mark.parametrize("rows,cols", [(1, 8), (5, 72), (128, 256), (130, 264), (300, 1000), (257, 1096), (64, 4104)])
def test_residual_and_lfull_error_ragged_shapes(ctx, oracle, rows, cols):
    ctx.reserve(rows, cols)
    ctx.apply_scale(None)
    w, g = inputs.make_rows(rows, cols, 40 + cols)
    H = inputs.make_gram(cols, 50 + cols)
    res = oracle.cluster_rows(w, g, BITS, 10, want_codes=False)
    c32 = res["centroids"].astype(np.float32)
    W, Cc = torch.from_numpy(w).cuda(), torch.from_numpy(c32).cuda()
    for b in BITS:
        D = oracle.residual(w, c32, BITS, width=b, exp2=8)
        Dg = ctx.residual(W, Cc, BITS, width=b, exp2=8)
        np.testing.assert_array_equal(Dg.cpu().numpy().view(np.uint16), D.view(np.uint16))
        if b in (1, 4):
            _check_err(ctx, oracle, D, H, 8, label=f"{rows}x{cols} b={b}")


def test_residual_with_scale_and_row_widths(ctx, oracle):
    rows, cols = 37, 520
    w, g = inputs.make_rows(rows, cols, 61)
    s = inputs.make_scale(cols, 62)
    bits = (np.arange(rows) * 3 % 4 + 1).astype(np.uint8)
    ctx.reserve(rows, cols)
    ctx.apply_scale(torch.from_numpy(s).cuda())
    res = oracle.cluster_rows(w, g, BITS, 12, s=s, want_codes=False)
    c32 = res["centroids"].astype(np.float32)
    for e in (0, 6, 11):
        D = oracle.residual(w, c32, BITS, row_bits=bits, s=s, exp2=e)
        Dg = ctx.residual(torch.from_numpy(w).cuda(), torch.from_numpy(c32).cuda(), BITS, row_bits=torch.from_numpy(bits).cuda(),
                          s=torch.from_numpy(s).cuda(), exp2=e)
        np.testing.assert_array_equal(Dg.cpu().numpy().view(np.uint16), D.view(np.uint16))
    assert ctx.get_status() == 0
    # alpha given although none is installed (or the reverse) is an argument error; a width outside the set a status bit
    ctx.apply_scale(None)
    from paper_2412_04180_b200.skim import SkimError
    with pytest.raises(SkimError) as e:
        ctx.residual(torch.from_numpy(w).cuda(), torch.from_numpy(c32).cuda(), BITS, width=2, s=torch.from_numpy(s).cuda())
    assert e.value.code == -8
    bad = bits.copy()
    bad[3] = 7
    ctx.residual(torch.from_numpy(w).cuda(), torch.from_numpy(c32).cuda(), BITS, row_bits=torch.from_numpy(bad).cuda())
    assert ctx.get_status() == 8


def test_lfull_special_matrices(ctx, oracle):
    """Zero residual rows give exactly zero; a diagonal H gives sum h d^2; an integer Gram matrix gives |d X|^2."""
    rows, cols = 140, 512
    rng = np.random.default_rng(7)
    ctx.reserve(rows, cols)
    D = (rng.standard_normal((rows, cols)) * 2).astype(np.float16)
    D[5] = 0
    D[77, 100:] = 0
    h = np.exp(rng.standard_normal(cols)).astype(np.float16)
    Hd = np.diag(h.astype(np.float64)).astype(np.float16)
    got = _check_err(ctx, oracle, D, Hd, 0, label="diagonal")
    assert got[5] == 0.0
    np.testing.assert_allclose(got, (D.astype(np.float64) ** 2 * h.astype(np.float64)).sum(axis=1), rtol=1e-5)
    X = rng.integers(-1, 2, size=(cols, 48)).astype(np.float64)
    Hx = (X @ X.T).astype(np.float16)
    got = _check_err(ctx, oracle, D, Hx, 0, label="integer gram")
    want = ((D.astype(np.float64) @ X) ** 2).sum(axis=1)
    np.testing.assert_allclose(got, want, rtol=1e-4, atol=1e-3)
    # power-of-two scaling of the residual is undone exactly by exp2
    got2 = ctx.err_lfull(torch.from_numpy((D.astype(np.float32) * 4).astype(np.float16)).cuda(), torch.from_numpy(Hx).cuda(), exp2=2)
    got3 = ctx.err_lfull(torch.from_numpy(D).cuda(), torch.from_numpy(Hx).cuda(), exp2=0)
    assert torch.equal(got2, got3)


@pytest.mark.parametrize("cols", [968, 1160, 2560])
def test_lfull_error_full_and_split_rounds(ctx, oracle, cols):
    """4096 rows are 32 row tiles.  On a 148-SM part 968 columns give 128 tiles (one round, nothing cut), 1160
    columns 160 tiles (one full round, the 12 tiles left cut into 8 ranges of K each), 2560 columns 320 tiles (two
    full rounds, 24 tiles cut into 6 ranges): rows from full tiles and from cut tiles are compared with the oracle."""
    rows = 4096
    ctx.reserve(rows, cols)
    rng = np.random.default_rng(cols)
    D = (rng.standard_normal((rows, cols)) * 0.25).astype(np.float16)
    H = inputs.make_gram(cols, 900 + cols)
    sample = np.sort(rng.choice(rows, size=200, replace=False))
    sample[0], sample[-1] = 0, rows - 1
    _check_err(ctx, oracle, D, H, 0, rows=sample, label=f"cols={cols}")


@pytest.mark.parametrize("cols,rows_total,seed", [(4096, 4096, 2000), (11008, 4096, 3001)])
def test_lfull_table_at_llama_shapes(ctx, oracle, cols, rows_total, seed):
    """The L-full error table of a full-size matrix (the launch configuration the benchmark times), all four
    widths from the GPU's own clustering; the oracle evaluates a sample of rows of every width column, and the
    greedy allocation over the table keeps its selection property."""
    rows = rows_total
    w, g = inputs.make_matrix(rows, cols, seed)
    H = inputs.make_gram(cols, seed + 7)
    ctx.reserve(rows, cols)
    ctx.apply_scale(None)
    W, G, Hc = torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda(), torch.from_numpy(H).cuda()
    cent, _, err_diag = ctx.cluster_rows(W, G, BITS, 50)
    table = torch.empty((rows, 4), dtype=torch.float32, device="cuda")
    scratch = torch.empty(ctx.err_lfull_bytes(rows, cols), dtype=torch.uint8, device="cuda")
    Dbuf = torch.empty((rows, cols), dtype=torch.float16, device="cuda")
    sample = np.sort(np.random.default_rng(cols).choice(rows, size=6, replace=False))
    c32 = cent.cpu().numpy()
    for bi, b in enumerate(BITS):
        ctx.residual(W, cent, BITS, width=b, out=Dbuf)
        ctx.err_lfull(Dbuf, Hc, scratch=scratch, out=table[:, bi], out_stride=4)
        torch.cuda.synchronize()
        Dh = Dbuf[torch.from_numpy(sample).cuda()].cpu().numpy()
        np.testing.assert_array_equal(Dh.view(np.uint16), oracle.residual(w[sample], c32[sample], BITS, width=b).view(np.uint16))
        want, mag = oracle.err_lfull(Dh, H)
        got = table[:, bi].cpu().numpy().astype(np.float64)[sample]
        assert np.all(np.abs(got - want) <= _bound(cols, mag))
        assert np.all(np.abs(got - want) <= 64 * 2.0 ** -24 * mag)
    assert ctx.get_status() == 0
    t = table.cpu().numpy()
    assert np.all(np.isfinite(t)) and np.all(t >= 0)
    assert np.mean(t[:, 0] > t[:, 3]) > 0.999
    bits, total = ctx.allocate_bits(table, BITS, 3.0)
    assert total == 3 * rows == int(bits.sum().item())
    from test_gpu_pipeline import _check_greedy_selection
    _check_greedy_selection(t, bits.cpu().numpy())
    # and bit-exact against the sequential greedy on the same table
    want_bits, _ = oracle.allocate_bits(t, 1, 3.0)
    np.testing.assert_array_equal(bits.cpu().numpy(), want_bits)


def test_lfull_argument_errors(ctx, skimlib):
    ctx.reserve(16, 64)
    D = torch.zeros((16, 64), dtype=torch.float16, device="cuda")
    H = torch.zeros((64, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(skimlib.SkimError) as e:
        ctx.err_lfull(D[:, :60].contiguous(), H[:60, :60].contiguous())       # cols % 8 != 0
    assert e.value.code == -2
    with pytest.raises(skimlib.SkimError) as e:
        ctx.err_lfull(D, H, scratch=torch.empty(256, dtype=torch.uint8, device="cuda")[:16])
    assert e.value.code == -5
    with pytest.raises(skimlib.SkimError) as e:
        ctx.err_lfull(D, H, exp2=40)
    assert e.value.code == -2
    assert float(ctx.err_lfull(D, H).abs().max().item()) == 0.0
