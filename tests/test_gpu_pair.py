"""The Winograd contraction on pairs of SMs (256 x 256 blocks per work item, tcgen05.mma.cta_group::2): layers with at
least 256 output channels and enough work items take it.  Element-wise parity with the CPU oracle on shapes that
leave the last 256-row block ragged (one CTA of the pair with a partial or empty tile), a ragged last channel
block, all operand formats (hi + lo pairs fetched with one copy, single-pass operands with 128-byte rows), and an
integer run that must be exact."""
import numpy as np
import pytest

from oracle import direct_conv as oc
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import assert_close, to_dev

pytestmark = pytest.mark.gpu

OPERANDS = {"bf16": B.OPERAND_BF16, "tf32": B.OPERAND_TF32}


def run(torch, layer, opts, inputs):
    x, w, b = inputs
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad, layer.dilation,
                          opts)
    y = r.run(to_dev(torch, x), to_dev(torch, w), to_dev(torch, b))
    torch.cuda.synchronize()
    assert r.device_status() == 0
    out = y.cpu().numpy()
    r.close()
    return out


# (N, Cin, Cout, H, k, m, operand, passes): work items = ceil(tiles / 256) * ceil(Cout / 256) * alpha^2 >= 148
@pytest.mark.parametrize("N,Cin,Cout,H,k,m,operand,passes", [
    (24, 256, 256, 28, 3, 4, "bf16", 3),      # 1176 tiles: the fifth row block holds 128 + 24 rows
    (8, 64, 300, 40, 5, 4, "tf32", 3),        # two channel blocks, the second of 44 channels; TF32 hi + lo
    (12, 128, 512, 30, 3, 2, "tf32", 1),      # single-pass TF32, 2700 tiles: the last block's second CTA is empty
    (10, 128, 256, 48, 3, 2, "bf16", 1),      # single-pass BF16 (128-byte rows of 64 elements)
    (6, 64, 288, 44, 3, 4, "bf16", 3),        # 288 channels: a second block of 32, 121 tiles per image
])
def test_pair_contraction_parity(N, Cin, Cout, H, k, m, operand, passes):
    import torch
    assert torch.cuda.is_available()
    B.lib()
    layer = W.ConvLayer("t", N, Cin, Cout, H, H, k, 1, (k - 1) // 2, 1, relu=True, seed=Cin + Cout + H)
    inputs = W.make_inputs(layer)
    opts = B.make_opts(relu=True, force_algo=B.ALGO_WINOGRAD, force_m=m, operand=OPERANDS[operand], passes=passes)
    got = run(torch, layer, opts, inputs)
    ref = oc.direct_conv(*inputs, 1, (k - 1) // 2, 1, 1, True)
    exact_enough = passes == 3 or (operand == "tf32" and m == 2)
    assert_close(got, ref, B.PREC_TF32 if exact_enough else B.PREC_BF16, "pair contraction")


def test_pair_contraction_exact_on_integers():
    """Small integers and F(2x2,3x3) with unit points (transform entries are multiples of 1/4): every product and sum
    is exact in TF32 and fp32, so the result must equal the oracle's bit for bit, in two runs."""
    import torch
    B.lib()
    layer = W.ConvLayer("t", 12, 64, 256, 30, 30, 3, 1, 1, 1, relu=False, seed=5)
    inputs = W.integer_inputs(layer, -2, 2)
    opts = B.make_opts(relu=False, force_algo=B.ALGO_WINOGRAD, force_m=2, operand=B.OPERAND_TF32, passes=1, points_id=2)
    ref = oc.direct_conv(*inputs, 1, 1, 1, 1, False)
    for _ in range(2):
        got = run(torch, layer, opts, inputs)
        assert np.array_equal(got.astype(np.float64), ref)

def test_pair_contraction_in_chunks():
    """A run split into chunks of images whose last chunk is smaller: the pair kernel then gets fewer tiles than its
    tensor maps were made for, and every chunk must still equal the oracle."""
    import torch
    B.lib()
    layer = W.ConvLayer("t", 25, 64, 256, 40, 40, 3, 1, 1, 1, relu=True, seed=11)
    inputs = W.make_inputs(layer)
    opts = B.make_opts(relu=True, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=B.OPERAND_BF16, passes=3, chunk_images=11)
    got = run(torch, layer, opts, inputs)                 # chunks of 11, 11 and 3 images: 1100 / 1100 / 300 tiles (180 work items per full chunk)
    ref = oc.direct_conv(*inputs, 1, 1, 1, 1, True)
    assert_close(got, ref, B.PREC_TF32, "pair contraction in chunks")
