"""The GEMM scheme without a patch matrix (producer warps gather the patches inside the tensor-core kernel)
against the fp64 direct-convolution oracle, through the C ABI."""
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


def run(torch, layer, inputs=None):
    x, w, b = inputs if inputs is not None else W.make_inputs(layer)
    o = B.make_opts(relu=layer.relu, force_algo=B.ALGO_GEMM, gemm_lhs=B.GEMM_LHS_IMPLICIT)
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad, layer.dilation, o)
    info = r.info
    assert info.algo == B.ALGO_GEMM and info.gemm_lhs == B.GEMM_LHS_IMPLICIT and info.v_bytes == 0
    assert info.launches_per_run == 1 and (info.operand, info.passes) == (B.OPERAND_TF32, 1)
    y = torch.full((layer.N, layer.Cout, info.OH, info.OW), float("nan"), device="cuda:0")
    r.run(to_dev(torch, x), to_dev(torch, w), to_dev(torch, b), y)
    torch.cuda.synchronize()
    assert r.device_status() == 0
    out = y.cpu().numpy()
    r.close()
    return out, (x, w, b)


def oracle(layer, x, w, b):
    return oc.direct_conv(x, w, b, layer.stride, layer.pad, layer.dilation, 1, layer.relu)


# (N, Cin, Cout, H, W, k, stride, pad, dilation)
SHAPES = [
    (2, 3, 64, 32, 32, 7, 2, 3, 1),        # stem: three input channels, K = 147
    (2, 64, 128, 20, 20, 3, 2, 1, 1),      # 3x3 stride 2
    (3, 24, 40, 13, 11, 3, 1, 1, 2),       # dilation 2
    (2, 16, 300, 9, 9, 3, 2, 0, 1),        # two channel blocks, no padding
    (1, 64, 128, 15, 15, 1, 2, 0, 1),      # 1x1 stride-2 downsample
    (4, 40, 24, 7, 7, 1, 1, 0, 1),         # pointwise on 7 x 7 (H*W not a multiple of 4)
    (1, 8, 8, 5, 5, 5, 1, 2, 1),           # 5x5, fewer positions than a tile
    (2, 20, 33, 10, 12, 2, 1, 1, 1),       # even kernel, odd channel counts
    (1, 7, 9, 9, 9, 3, 3, 2, 2),           # stride 3, pad 2, dilation 2
]


@pytest.mark.parametrize("shape", SHAPES)
def test_parity(torch, shape):
    N, Cin, Cout, H, W_, k, s, p, d = shape
    layer = W.ConvLayer("ig", N, Cin, Cout, H, W_, k, s, p, d, relu=True, x_dist="normal", w_dist="kaiming", seed=sum(shape))
    got, (x, w, b) = run(torch, layer)
    assert_close(got, oracle(layer, x, w, b), B.PREC_TF32, "implicit GEMM")


@pytest.mark.parametrize("shape", SHAPES[:5])
def test_integer_inputs_bit_exact(torch, shape):
    N, Cin, Cout, H, W_, k, s, p, d = shape
    layer = W.ConvLayer("ig", N, Cin, Cout, H, W_, k, s, p, d, relu=False, seed=11)
    x, w, b = W.integer_inputs(layer, -3, 3)
    got, _ = run(torch, layer, inputs=(x, w, b))
    assert np.array_equal(got.astype(np.float64), oracle(layer, x, w, b))


def test_resnet_stem_full_size_sampled(torch):
    layer = W.config2(32)[0]
    x, w, b = W.make_inputs(layer)
    got, _ = run(torch, layer, inputs=(x, w, b))
    rng = np.random.Generator(np.random.PCG64(5))
    idx = rng.integers(0, got.size, size=8192)
    ref = oc.direct_conv_at(x, w, b, idx, layer.stride, layer.pad, layer.dilation, 1, layer.relu)
    assert_close(got.ravel()[idx], ref, B.PREC_TF32, "stem samples")
    first = got.copy()
    again, _ = run(torch, layer, inputs=(x, w, b))
    assert np.array_equal(first, again)


def test_where_it_does_not_apply(torch):
    with pytest.raises(B.MnnError):      # BF16 operands
        B.mnn_conv_plan_ex(1, 16, 16, 8, 8, 3, 2, 1, 1, B.make_opts(force_algo=B.ALGO_GEMM, gemm_lhs=B.GEMM_LHS_IMPLICIT,
                                                                    operand=B.OPERAND_BF16))
    with pytest.raises(B.MnnError):      # grouped
        B.mnn_conv_plan_ex(1, 16, 16, 8, 8, 3, 2, 1, 1, B.make_opts(groups=16, force_algo=B.ALGO_GEMM,
                                                                    gemm_lhs=B.GEMM_LHS_IMPLICIT))
