"""GPU parity of the single-kernel Winograd F(2x2, 3x3) path (input transform, tensor-core
contraction and output transform fused; Eq. 6) against the fp64 direct-convolution oracle,
through the C ABI.  Tolerance of the TF32 accuracy class: relative L2 <= 1e-3 and
max-abs <= 2e-2 * max|y_ref|; integer-valued inputs bit-exact."""
import numpy as np
import pytest

from oracle import direct_conv as oc
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import assert_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available()
    B.lib()
    return torch


def fused_opts(layer, **kw):
    return B.make_opts(groups=1, relu=layer.relu, fused=B.FUSED_ONLY, **kw)


def run_fused(torch, layer, inputs=None, **kw):
    x, w, b = inputs if inputs is not None else W.make_inputs(layer)
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, 3, 1, layer.pad, 1, fused_opts(layer, **kw))
    info = r.info
    assert info.fused == 1 and info.algo == B.ALGO_WINOGRAD and info.m == 2 and info.launches_per_run == 1
    assert info.v_bytes == 0 and info.m_bytes == 0 and info.chosen_candidate == 15
    xd, wd, bd = to_dev(torch, x), to_dev(torch, w), to_dev(torch, b)
    y = torch.full((layer.N, layer.Cout, info.OH, info.OW), float("nan"), device="cuda:0")
    r.run(xd, wd, bd, y)
    torch.cuda.synchronize()
    assert r.device_status() == 0
    out = y.cpu().numpy()
    r.close()
    return out, (x, w, b)


def oracle(layer, x, w, b):
    return oc.direct_conv(x, w, b, 1, layer.pad, 1, 1, layer.relu)


def test_config0(torch):
    layer = W.config0()[0]
    got, (x, w, b) = run_fused(torch, layer)
    assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, "config0 fused")


@pytest.mark.parametrize("batch", [1, 3])
@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config1_shapes(torch, batch, idx):
    layer = W.config1(batch)[idx]
    got, (x, w, b) = run_fused(torch, layer)
    assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, layer.name)


def test_config1_batch32_sampled(torch):
    # full size of the benchmark's second workload: first and last image in full, 4096 sampled outputs elsewhere
    for layer in W.config1(32):
        x, w, b = W.make_inputs(layer)
        got, _ = run_fused(torch, layer, inputs=(x, w, b))
        ref = oc.direct_conv_images(x, w, b, [0, layer.N - 1], 1, layer.pad, 1, 1, layer.relu)
        assert_close(got[[0, layer.N - 1]], ref, B.PREC_TF32, layer.name + " images")
        rng = np.random.Generator(np.random.PCG64(layer.seed + 9))
        idx = rng.integers(0, got.size, size=4096)
        ref_s = oc.direct_conv_at(x, w, b, idx, 1, layer.pad, 1, 1, layer.relu)
        assert_close(got.ravel()[idx], ref_s, B.PREC_TF32, layer.name + " samples")


@pytest.mark.parametrize("N,Cin,Cout,H,W_,pad", [
    (2, 8, 8, 7, 7, 1),          # ragged edges, fewer tiles than a block
    (1, 24, 40, 14, 14, 1),      # Cin not a multiple of 32, Cout not a multiple of 16
    (3, 40, 136, 13, 9, 1),      # odd output sizes, two channel blocks with a ragged second one
    (2, 64, 72, 33, 20, 0),      # no padding, even OW
    (1, 16, 16, 6, 10, 2),       # pad 2: outputs larger than the input
    (5, 32, 200, 5, 5, 1),       # 3 x 3 tiles per image: blocks straddle images
    (2, 3, 16, 12, 12, 1),       # three input channels (one partly filled K block)
    (1, 21, 33, 9, 9, 1),        # odd channel counts on both sides
])
def test_odd_shapes(torch, N, Cin, Cout, H, W_, pad):
    layer = W.ConvLayer("t", N, Cin, Cout, H, W_, 3, 1, pad, relu=True, x_dist="normal", w_dist="kaiming", seed=N * 7 + Cin)
    got, (x, w, b) = run_fused(torch, layer)
    assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, "odd shape")


@pytest.mark.parametrize("pid", [B.POINTS_PAPER, B.POINTS_UNIT, B.POINTS_MIXED])
def test_integer_inputs_bit_exact(torch, pid):
    # small integers: every product and partial sum is exact in TF32 / fp32, for every point set whose
    # matrices are dyadic (all three are at alpha = 4)
    layer = W.ConvLayer("t", 2, 48, 160, 12, 14, 3, 1, 1, relu=False, seed=31)
    x, w, b = W.integer_inputs(layer, -2, 2)
    kw = dict(points_id=pid, operand=B.OPERAND_TF32, passes=1, force_m=2)
    got, _ = run_fused(torch, layer, inputs=(x, w, b), **kw)
    ref = oracle(layer, x, w, b)
    assert np.array_equal(got.astype(np.float64), ref)


def test_zero_input_gives_relu_of_bias(torch):
    layer = W.ConvLayer("t", 2, 32, 48, 10, 10, 3, 1, 1, relu=True, seed=3)
    x, w, b = W.make_inputs(layer)
    x[:] = 0
    got, _ = run_fused(torch, layer, inputs=(x, w, b))
    want = np.broadcast_to(np.maximum(b, 0)[None, :, None, None], got.shape)
    assert np.array_equal(got, want)


def test_repeatable(torch):
    layer = W.config1(3)[1]
    x, w, b = W.make_inputs(layer)
    first, _ = run_fused(torch, layer, inputs=(x, w, b))
    for _ in range(9):
        again, _ = run_fused(torch, layer, inputs=(x, w, b))
        assert np.array_equal(first, again)


def test_where_it_does_not_apply(torch):
    for args, kw in (((1, 16, 16, 8, 8, 3, 2, 1, 1), {}),          # stride 2
                     ((1, 16, 16, 8, 8, 5, 1, 2, 1), {}),          # 5x5
                     ((1, 16, 16, 8, 8, 3, 1, 1, 1), {"operand": B.OPERAND_BF16})):
        with pytest.raises(B.MnnError):
            B.mnn_conv_plan_ex(*args, B.make_opts(fused=B.FUSED_ONLY, **kw))
