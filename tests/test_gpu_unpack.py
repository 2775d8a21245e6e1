"""GPU parity of the unpacking kernels against the oracle.  The GPU stages are fed the ORACLE's
packed words, row order, group tables and codebooks; nothing the CUDA path produced reaches the
oracle.  skim_dequantize is bit-exact; skim_matvec accumulates in binary32 and must stay within
(cols/32 + 8) * 2^-24 * sum |terms| of the oracle's binary64 sum (the recursive-summation bound for
the kernel's accumulation order)."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs

pytestmark = pytest.mark.gpu


def _synthetic_emit(oracle, rows, cols, bit_set, seed, scaled, widths=None):
    """Oracle packing of a synthetic matrix with random ascending codebooks (no clustering needed)."""
    w, _ = inputs.make_rows(rows, cols, seed)
    rng = np.random.default_rng(seed)
    sumk = sum(1 << b for b in bit_set)
    cent = np.concatenate([np.sort(rng.standard_normal((rows, 1 << b)).astype(np.float32) * 0.03, axis=1)
                           for b in bit_set], axis=1)
    assert cent.shape == (rows, sumk)
    if widths is None:
        widths = rng.choice(bit_set, size=rows)
    bits = np.asarray(widths, dtype=np.uint8)
    s = inputs.make_scale(cols, seed + 1) if scaled else None
    em = oracle.emit(w, bits, cent, bit_set, s=s)
    return em, s


def _to_gpu(em):
    max_words = max(4, em["packed"].size)
    packed = np.zeros(max_words, np.uint32)
    packed[:em["packed"].size] = em["packed"]
    return dict(packed=torch.from_numpy(packed.view(np.int32)).cuda(),
                row_order=torch.from_numpy(em["row_order"]).cuda(),
                group_info=torch.from_numpy(np.concatenate([em["group_start"], em["group_word"]])).cuda(),
                lut=torch.from_numpy(em["lut"].view(np.int16)).cuda())


def _check(ctx, oracle, em, s, cols, bit_set, seed, padded_out=False):
    q = _to_gpu(em)
    rows = em["row_order"].size
    sd = torch.from_numpy(s).cuda() if s is not None else None
    want = oracle.dequantize(em, cols, bit_set, s=s)
    if padded_out:
        buf = torch.full((rows, cols + 3), -7.0, dtype=torch.float16, device="cuda")
        out = ctx.dequantize(q, cols, bit_set, s=sd, out=buf[:, :cols])
        assert torch.all(buf[:, cols:] == -7.0)                # nothing written past the row
    else:
        out = ctx.dequantize(q, cols, bit_set, s=sd)
    np.testing.assert_array_equal(out.cpu().numpy().view(np.uint16), want.view(np.uint16))
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(cols).astype(np.float16)
    y_want, mag = oracle.matvec(em, cols, bit_set, x, s=s)
    y = ctx.matvec(q, cols, bit_set, torch.from_numpy(x).cuda(), s=sd).cpu().numpy().astype(np.float64)
    bound = (cols / 32 + 8) * 2.0 ** -24 * mag + 1e-45
    assert np.all(np.abs(y - y_want) <= bound), float(np.max(np.abs(y - y_want) / bound))


@pytest.mark.parametrize("cols", [1, 7, 8, 31, 32, 33, 255, 256, 257, 1000, 4096, 5000])
@pytest.mark.parametrize("scaled", [False, True])
def test_unpack_matches_oracle_on_ragged_widths(ctx, oracle, cols, scaled):
    em, s = _synthetic_emit(oracle, 37, cols, [1, 2, 3, 4], 700 + cols, scaled)
    _check(ctx, oracle, em, s, cols, [1, 2, 3, 4], cols)


@pytest.mark.parametrize("bit_set", [[1], [2, 3], [3], [3, 4], [4], [1, 2, 3]])
def test_unpack_other_bit_sets_and_unaligned_output(ctx, oracle, bit_set):
    em, s = _synthetic_emit(oracle, 65, 777, bit_set, 31 + len(bit_set), True)
    _check(ctx, oracle, em, s, 777, bit_set, 5, padded_out=True)


def test_unpack_empty_groups_and_single_rows(ctx, oracle):
    for widths in ([4] * 33, [1] * 5, [2], [3, 3, 1]):
        em, s = _synthetic_emit(oracle, len(widths), 300, [1, 2, 3, 4], 11, True, widths=widths)
        _check(ctx, oracle, em, s, 300, [1, 2, 3, 4], 3)


@pytest.mark.parametrize("rows,cols", [(600, 11008), (1500, 4096), (200, 22016)])
def test_unpack_llama_row_lengths(ctx, oracle, rows, cols):
    em, s = _synthetic_emit(oracle, rows, cols, [1, 2, 3, 4], 40 + rows, True)
    _check(ctx, oracle, em, s, cols, [1, 2, 3, 4], rows)


def test_unpack_after_the_real_pipeline(ctx, oracle):
    """The consumer kernels on what the GPU pipeline itself packed: labels decoded by the dequantiser
    are the midpoint-count labels of the GPU's own centroids (checked in numpy)."""
    rows, cols = 256, 512
    w, g = inputs.make_matrix(rows, cols, 0)
    ctx.reserve(rows, cols)
    W, G = torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda()
    cent, _, err = ctx.cluster_rows(W, G, [1, 2, 3, 4], 30)
    bits, _ = ctx.allocate_bits(err, [1, 2, 3, 4], 3.2)
    q = ctx.quantize(W, bits, cent, [1, 2, 3, 4])
    wq = ctx.dequantize(q, cols, [1, 2, 3, 4]).cpu().numpy()
    c, b = cent.cpu().numpy(), bits.cpu().numpy()
    offs = {1: 0, 2: 2, 3: 6, 4: 14}
    for i in range(0, rows, 7):
        k = 1 << int(b[i])
        ci = c[i, offs[int(b[i])]:offs[int(b[i])] + k].astype(np.float64)
        mid = 0.5 * (ci[:-1] + ci[1:])
        labels = (mid[None, :] < w[i].astype(np.float64)[:, None]).sum(axis=1)
        np.testing.assert_array_equal(wq[i].view(np.uint16), ci.astype(np.float32).astype(np.float16)[labels].view(np.uint16))


def test_unpack_argument_errors(ctx, oracle, skimlib):
    em, s = _synthetic_emit(oracle, 8, 64, [1, 2, 3, 4], 1, False)
    q = _to_gpu(em)
    with pytest.raises(skimlib.SkimError) as e:
        ctx.dequantize(q, 64, [1, 3])
    assert e.value.code == -3
    with pytest.raises(skimlib.SkimError) as e:
        ctx.dequantize(q, 0, [1, 2, 3, 4], out=torch.empty((8, 64), dtype=torch.float16, device="cuda"))
    assert e.value.code == -2
    with pytest.raises(skimlib.SkimError) as e:
        ctx.matvec(q, 100000, [1, 2, 3, 4], torch.zeros(100000, dtype=torch.float16, device="cuda"))
    assert e.value.code == -2
