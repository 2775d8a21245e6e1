"""skim_quantize_static: the packer for callers that are not allowed to allocate device memory
(plugin or allocator callbacks, processes with a fixed device-memory plan).  It must give exactly
what skim_quantize gives, call after call, although every call reuses one built-in scratch array.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from paper_2412_04180_b200 import inputs

pytestmark = pytest.mark.gpu
BITS = [1, 2, 3, 4]


def _outputs(skimlib, rows, cols):
    _, mx = skimlib.Skim.packed_layout(rows, cols, BITS)
    return dict(packed=torch.zeros(mx // 4, dtype=torch.int32, device="cuda"),
                row_order=torch.zeros(rows, dtype=torch.int32, device="cuda"),
                group_info=torch.zeros(10, dtype=torch.int64, device="cuda"),
                lut=torch.zeros((rows, 16), dtype=torch.int16, device="cuda"))


def _same(a, b):
    words = int(a["group_info"][-1].item())
    assert words == int(b["group_info"][-1].item()) and words > 0
    nb = (a["group_info"].numel() - 2) // 2
    placed = int(a["group_info"][nb].item())      # rows with a valid width; entries beyond are not written
    assert torch.equal(a["group_info"], b["group_info"])
    assert torch.equal(a["row_order"][:placed], b["row_order"][:placed])
    order = a["row_order"][:placed].long()
    assert torch.equal(a["lut"][order], b["lut"][order])
    assert torch.equal(a["packed"][:words], b["packed"][:words])


def test_static_variant_matches_skim_quantize_on_two_calls_in_a_row(skimlib):
    from paper_2412_04180_b200.skim import Skim, quantize_static
    ctx = Skim(device=0)
    # first call: a larger matrix, so that the scratch is left full of stale positions
    rows1, cols1 = 700, 1000
    w1, g1 = inputs.make_rows(rows1, cols1, 901)
    ctx.reserve(rows1, cols1)
    W1, G1 = torch.from_numpy(w1).cuda(), torch.from_numpy(g1).cuda()
    cent1, _, err1 = ctx.cluster_rows(W1, G1, BITS, 8)
    bits1, _ = ctx.allocate_bits(err1, BITS, 2.6)
    ref1 = ctx.quantize(W1, bits1, cent1, BITS)
    out1 = _outputs(skimlib, rows1, cols1)
    torch.cuda.synchronize()
    quantize_static(W1, bits1, cent1, BITS, out1)
    torch.cuda.synchronize()
    _same(out1, ref1)

    # second call right after: fewer rows, other widths (one of them invalid), another shape
    rows2, cols2 = 123, 517
    w2, g2 = inputs.make_rows(rows2, cols2, 902)
    W2, G2 = torch.from_numpy(w2).cuda(), torch.from_numpy(g2).cuda()
    cent2, _, err2 = ctx.cluster_rows(W2, G2, BITS, 8)
    bits2 = torch.from_numpy((np.arange(rows2) * 7 % 4 + 1).astype(np.uint8)).cuda()
    bits2[5] = 9
    ref2 = ctx.quantize(W2, bits2, cent2, BITS)
    assert ctx.get_status() == 8
    out2 = _outputs(skimlib, rows2, cols2)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    quantize_static(W2, bits2, cent2, BITS, out2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before        # nothing was allocated on the device
    _same(out2, ref2)
    assert int(out2["group_info"][4].item()) == rows2 - 1     # the invalid width was skipped

    # and the first problem again, after the smaller one
    out3 = _outputs(skimlib, rows1, cols1)
    quantize_static(W1, bits1, cent1, BITS, out3)
    torch.cuda.synchronize()
    _same(out3, ref1)
    ctx.close()


def test_static_variant_rejects_too_many_rows(skimlib):
    from paper_2412_04180_b200.skim import STATIC_MAX_ROWS, SkimError, quantize_static
    rows = STATIC_MAX_ROWS + 1
    W = torch.zeros((rows, 8), dtype=torch.float16, device="cuda")
    bits = torch.ones(rows, dtype=torch.uint8, device="cuda")
    cent = torch.zeros((rows, 30), device="cuda")
    with pytest.raises(SkimError, match="65536") as e:
        quantize_static(W, bits, cent, BITS, _outputs(skimlib, rows, 8))
    assert e.value.code == -10
