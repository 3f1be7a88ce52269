"""One recursion level of Strassen's algorithm on the 1x1-convolution matrix product (Section 3.3.2, Eq. 9)
against the fp64 direct-convolution oracle, through the C ABI; and the stopping rule against hand arithmetic."""
import numpy as np
import pytest

from oracle import direct_conv as oc
from oracle import planner_twin as T
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import assert_close, rel_l2, to_dev


def test_stopping_rule_matches_hand_arithmetic_and_the_twin():
    B.lib()
    # 256^3: saved 256^3 / 8 = 2097152 multiplications, added 15 * 128^2 = 245760 additions
    assert 256 ** 3 - 7 * 128 ** 3 == 2097152 and 15 * 128 ** 2 == 245760
    assert B.mnn_strassen_rule(256, 256, 256) == 1
    # saved = m n k / 8 for even sizes; with m = n = k = s the rule reads s^3 / 8 > 15 s^2 / 4, i.e. s > 30
    assert B.mnn_strassen_rule(30, 30, 30) == 0 and B.mnn_strassen_rule(32, 32, 32) == 1
    assert B.mnn_strassen_rule(1, 1000, 1000) == 0
    for m, n, k in [(2, 2, 2), (31, 33, 35), (512, 512, 1024), (8, 4096, 8), (1000, 3, 1000), (64, 64, 2)]:
        assert B.mnn_strassen_rule(m, n, k) == int(T.strassen_rule(m, n, k)), (m, n, k)


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available()
    B.lib()
    return torch


def run(torch, layer, inputs=None, **kw):
    x, w, b = inputs if inputs is not None else W.make_inputs(layer)
    o = B.make_opts(relu=layer.relu, strassen=1, **kw)
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, 1, 1, 0, 1, o)
    assert r.info.strassen == 1 and r.info.algo == B.ALGO_GEMM and r.info.launches_per_run == 3
    y = r.run(to_dev(torch, x), to_dev(torch, w), to_dev(torch, b))
    torch.cuda.synchronize()
    assert r.device_status() == 0
    out = y.cpu().numpy()
    info = r.info
    r.close()
    return out, info, (x, w, b)


@pytest.mark.gpu
@pytest.mark.parametrize("N,Cin,Cout,H", [(2, 64, 64, 8), (4, 96, 40, 7), (2, 18, 6, 5), (6, 256, 130, 14), (2, 512, 512, 16)])
@pytest.mark.parametrize("prec", [B.PREC_TF32, B.PREC_BF16])
def test_parity(torch, N, Cin, Cout, H, prec):
    layer = W.ConvLayer("s", N, Cin, Cout, H, H, 1, 1, 0, relu=True, x_dist="normal", w_dist="kaiming", seed=N + Cin)
    got, info, (x, w, b) = run(torch, layer, precision=prec)
    ref = oc.direct_conv(x, w, b, 1, 0, 1, 1, True)
    assert_close(got, ref, prec, "strassen")
    if prec == B.PREC_TF32:
        assert (info.operand, info.passes) == (B.OPERAND_BF16, 3) and rel_l2(got, ref) < 5e-5


@pytest.mark.gpu
@pytest.mark.parametrize("operand,passes", [(B.OPERAND_TF32, 1), (B.OPERAND_BF16, 1), (B.OPERAND_BF16, 3), (B.OPERAND_TF32, 3)])
def test_integer_inputs_bit_exact(torch, operand, passes):
    layer = W.ConvLayer("s", 4, 48, 24, 9, 9, 1, 1, 0, relu=False, seed=5)
    x, w, b = W.integer_inputs(layer, -3, 3)
    got, _, _ = run(torch, layer, inputs=(x, w, b), operand=operand, passes=passes)
    assert np.array_equal(got.astype(np.float64), oc.direct_conv(x, w, b, 1, 0, 1, 1, False))


@pytest.mark.gpu
def test_where_it_does_not_apply(torch):
    for args in ((3, 64, 64, 8, 8, 1, 1, 0, 1), (2, 63, 64, 8, 8, 1, 1, 0, 1), (2, 64, 64, 8, 8, 3, 1, 1, 1),
                 (2, 64, 64, 8, 8, 1, 2, 0, 1)):
        with pytest.raises(B.MnnError):
            B.mnn_conv_plan_ex(*args, B.make_opts(strassen=1))
