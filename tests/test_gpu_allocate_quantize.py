"""GPU parity: the allocator and the packer are bit-exact against the oracle when both sides are
fed the same error table / the same widths and binary32 centroids."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs
from parity import unpack_row

pytestmark = pytest.mark.gpu
BITS = [1, 2, 3, 4]


def _alloc(ctx, err, bit_set, budget):
    bits, total = ctx.allocate_bits(torch.from_numpy(err).cuda(), bit_set, budget)
    return bits.cpu().numpy(), total


@pytest.mark.parametrize("monotone", [True, False])
@pytest.mark.parametrize("ties", [False, True])
@pytest.mark.parametrize("rows", [1, 2, 31, 256, 1000, 4096])
def test_allocation_matches_sequential_greedy(ctx, oracle, rows, monotone, ties):
    err = inputs.make_error_table(rows, 4, 100 + rows, monotone=monotone, ties=ties)
    for budget in (1.0, 1.3, 2.25, 2.5, 3.0, 3.2, 3.999, 4.0):
        want, total = oracle.allocate_bits(err, 1, budget)
        got, gtotal = _alloc(ctx, err, BITS, budget)
        assert gtotal == total
        np.testing.assert_array_equal(got, want, err_msg=f"rows={rows} budget={budget}")
        assert int(got.sum()) == total


def test_allocation_heavy_ties_and_special_tables(ctx, oracle):
    rng = np.random.default_rng(4)
    tables = [
        np.zeros((300, 4), np.float32),                                   # every reduction equal (zero)
        np.tile(np.array([[8, 4, 2, 1]], np.float32), (257, 1)),         # identical rows
        rng.integers(0, 3, size=(500, 4)).astype(np.float32),            # many exact ties, negative gains
        np.array([[12, 2, 1, 0], [9, 5, 2, 0], [9, 5, 0, 0]], np.float32),
        np.array([[1, 2, 3, 4], [5, 1, 2, 9]], np.float32),              # more bits make it worse
        np.abs(rng.standard_normal((64, 4))).astype(np.float32) * np.float32(1e-30),   # tiny values
        np.abs(rng.standard_normal((64, 4))).astype(np.float32) * np.float32(1e30),    # huge values
    ]
    for t, err in enumerate(tables):
        n = err.shape[0]
        for total in sorted(set([n, n + 1, n + n // 2, 2 * n, 2 * n + 1, 3 * n - 1, 3 * n, 4 * n - 1, 4 * n])):
            budget = total / n
            want, tot = oracle.allocate_bits(err, 1, budget)
            got, gtot = _alloc(ctx, err, BITS, budget)
            assert gtot == tot
            np.testing.assert_array_equal(got, want, err_msg=f"table {t} total {total}")


@pytest.mark.parametrize("rows", [1, 33, 1000, 4096, 9000])
def test_floor_started_allocation_matches_oracle(ctx, oracle, rows):
    """skim_allocate_bits_floor: every row starts at floor(budget); bit-exact against the oracle's loop."""
    err = inputs.make_error_table(rows, 4, 300 + rows, monotone=False, ties=True)
    errd = torch.from_numpy(err).cuda()
    for budget in (1.0, 1.25, 2.0, 2.25, 2.999, 3.0, 3.5, 4.0):
        want, total = oracle.allocate_bits(err, 1, budget, floor_start=True)
        got, gtotal = ctx.allocate_bits(errd, BITS, budget, floor_start=True)
        assert gtotal == total
        np.testing.assert_array_equal(got.cpu().numpy(), want, err_msg=f"rows={rows} budget={budget}")
    for bit_set in ([2, 3, 4], [3, 4]):
        sub = np.ascontiguousarray(err[:, :len(bit_set)])
        for budget in (bit_set[0] + 0.0, bit_set[0] + 0.6, bit_set[-1] - 0.3):
            want, total = oracle.allocate_bits(sub, bit_set[0], budget, floor_start=True)
            got, gtotal = ctx.allocate_bits(torch.from_numpy(sub).cuda(), bit_set, budget, floor_start=True)
            assert gtotal == total
            np.testing.assert_array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("rows", [1, 37, 1000, 5000])
def test_allocation_with_the_printed_stopping_rule_matches_oracle(ctx, oracle, rows):
    err = inputs.make_error_table(rows, 4, 900 + rows, monotone=False, ties=True)
    errd = torch.from_numpy(err).cuda()
    for budget in (1.0, 1.001, 2.25, 2.5003, 3.0, 3.9999, 4.0):
        want, total = oracle.allocate_bits(err, 1, budget, round_up=True)
        got, gtotal = ctx.allocate_bits(errd, BITS, budget, round_up=True)
        assert gtotal == total
        np.testing.assert_array_equal(got.cpu().numpy(), want, err_msg=f"rows={rows} budget={budget}")


@pytest.mark.parametrize("rows", [1, 7, 300, 2000])
def test_optimal_allocation_matches_oracle(ctx, oracle, rows):
    """skim_allocate_optimal: same recurrence, same order of additions, same tie rule as the oracle's dynamic
    programme, so widths and cost are bit-identical; the greedy never beats it."""
    err = inputs.make_error_table(rows, 4, 500 + rows, monotone=False, ties=True)
    errd = torch.from_numpy(err).cuda()
    for budget in (1.0, 1.4, 2.25, 3.0, 3.6, 4.0):
        want, total, cost = oracle.allocate_optimal(err, 1, budget)
        got, gtotal, gcost = ctx.allocate_optimal(errd, BITS, budget)
        assert gtotal == total and gcost == cost
        np.testing.assert_array_equal(got.cpu().numpy(), want, err_msg=f"rows={rows} budget={budget}")
        greedy, _ = ctx.allocate_bits(errd, BITS, budget)
        gsum = float(err[np.arange(rows), greedy.cpu().numpy().astype(np.int64) - 1].astype(np.float64).sum())
        assert gcost <= gsum * (1 + 1e-12) + 1e-300
    sub = np.ascontiguousarray(err[:, :2])
    want, total, cost = oracle.allocate_optimal(sub, 3, 3.5)
    got, gtotal, gcost = ctx.allocate_optimal(torch.from_numpy(sub).cuda(), [3, 4], 3.5)
    assert gtotal == total and gcost == cost
    np.testing.assert_array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("bit_set", [[2, 3], [1, 2, 3], [3, 4], [4]])
def test_allocation_other_bit_sets(ctx, oracle, bit_set):
    err = inputs.make_error_table(777, len(bit_set), 9, monotone=False, ties=True)
    for frac in (0.0, 0.37, 0.5, 1.0):
        budget = bit_set[0] + frac * (bit_set[-1] - bit_set[0])
        want, tot = oracle.allocate_bits(err, bit_set[0], budget)
        got, gtot = _alloc(ctx, err, bit_set, budget)
        assert gtot == tot
        np.testing.assert_array_equal(got, want)


def test_allocation_largest_row_count(ctx, oracle):
    err = inputs.make_error_table(22016, 4, 77, monotone=False)
    want, tot = oracle.allocate_bits(err, 1, 3.0)
    got, gtot = _alloc(ctx, err, BITS, 3.0)
    assert gtot == tot == 66048
    np.testing.assert_array_equal(got, want)


def test_allocation_budget_errors(ctx, skimlib):
    err = torch.zeros((10, 4), device="cuda")
    for budget in (0.99, 4.01, float("nan")):
        with pytest.raises(skimlib.SkimError) as e:
            ctx.allocate_bits(err, BITS, budget)
        assert e.value.code == -4


def _emit_both(ctx, oracle, w, bits, cent32, bit_set, s=None):
    rows, cols = w.shape
    ctx.reserve(rows, cols)
    ctx.apply_scale(torch.from_numpy(s).cuda() if s is not None else None)
    out = ctx.quantize(torch.from_numpy(w).cuda(), torch.from_numpy(bits).cuda(), torch.from_numpy(cent32).cuda(), bit_set)
    torch.cuda.synchronize()
    ctx.apply_scale(None)
    want = oracle.emit(w, bits, cent32, bit_set, s=s)
    nb = len(bit_set)
    info = out["group_info"].cpu().numpy()
    np.testing.assert_array_equal(info[:nb + 1], want["group_start"])
    np.testing.assert_array_equal(info[nb + 1:], want["group_word"])
    np.testing.assert_array_equal(out["row_order"].cpu().numpy(), want["row_order"])
    words = int(info[-1])
    np.testing.assert_array_equal(out["packed"].cpu().numpy().view(np.uint32)[:words], want["packed"])
    np.testing.assert_array_equal(out["lut"].cpu().numpy().view(np.uint16), want["lut"])
    return out, want


@pytest.mark.parametrize("cols", [1, 7, 8, 31, 32, 33, 100, 127, 128, 1000, 4096, 11008])
def test_packed_codes_are_bit_exact(ctx, oracle, cols):
    rows = 37
    w, g = inputs.make_rows(rows, cols, 300 + cols)
    cent32 = oracle.cluster_rows(w, g, BITS, 6, want_codes=False)["centroids"].astype(np.float32)
    bits = (np.arange(rows) * 3 % 4 + 1).astype(np.uint8)
    out, want = _emit_both(ctx, oracle, w, bits, cent32, BITS)
    # and the words decode back to the oracle's labels
    info = out["group_info"].cpu().numpy()
    packed = out["packed"].cpu().numpy().view(np.uint32)
    p = int(info[2])            # first packed row of the 3-bit group
    if info[3] > info[2]:
        stride = oracle.row_stride_words(cols, 3)
        row = want["row_order"][p]
        np.testing.assert_array_equal(unpack_row(packed[info[5 + 2]:info[5 + 2] + stride], cols, 3), want["codes"][row])


def test_packed_codes_with_scale_and_one_width_only(ctx, oracle):
    rows, cols = 19, 520
    w, g = inputs.make_rows(rows, cols, 8)
    s = inputs.make_scale(cols, 8)
    cent32 = oracle.cluster_rows(w, g, BITS, 6, s=s, want_codes=False)["centroids"].astype(np.float32)
    for b in BITS:
        _emit_both(ctx, oracle, w, np.full(rows, b, np.uint8), cent32, BITS, s=s)
    _emit_both(ctx, oracle, w, (np.arange(rows) % 4 + 1).astype(np.uint8), cent32, BITS, s=s)


def test_packed_codes_unaligned_leading_dimension(ctx, oracle):
    # cols not a multiple of 8: rows do not start on 16-byte boundaries (scalar load path)
    rows, cols = 11, 1003
    w, g = inputs.make_rows(rows, cols, 12)
    cent32 = oracle.cluster_rows(w, g, [2, 3], 6, want_codes=False)["centroids"].astype(np.float32)
    _emit_both(ctx, oracle, w, (np.arange(rows) % 2 + 2).astype(np.uint8), cent32, [2, 3])


def test_elements_exactly_at_midpoints(ctx, oracle):
    """Centroids chosen so that many elements sit exactly on a midpoint: they go to the lower cluster."""
    rows, cols = 4, 256
    w = (np.arange(rows * cols).reshape(rows, cols) % 33).astype(np.float16)       # integers 0..32
    cent = np.zeros((rows, 30), np.float32)
    cent[:, 0:2] = [8, 24]                            # midpoint 16
    cent[:, 2:6] = [4, 12, 20, 28]                    # midpoints 8, 16, 24
    cent[:, 6:14] = np.arange(8) * 4 + 2              # midpoints 4, 8, ...
    cent[:, 14:30] = np.arange(16) * 2 + 1            # midpoints 2, 4, ...
    cent[3, 14:30] = np.repeat(np.arange(8) * 4 + 2, 2)   # duplicate centroids
    bits = np.array([1, 2, 3, 4], np.uint8)
    _emit_both(ctx, oracle, w, bits, cent, BITS)
    _emit_both(ctx, oracle, w, np.array([4, 4, 4, 4], np.uint8), cent, BITS)


def test_quantize_flags_widths_outside_the_set(ctx, skimlib):
    w, g = inputs.make_rows(8, 64, 1)
    ctx.reserve(8, 64)
    bits = torch.tensor([1, 2, 3, 4, 5, 0, 2, 2], dtype=torch.uint8, device="cuda")
    cent = torch.zeros((8, 30), device="cuda")
    out = ctx.quantize(torch.from_numpy(w).cuda(), bits, cent, BITS)
    assert ctx.get_status() == 8
    assert int(out["group_info"][4]) == 6
