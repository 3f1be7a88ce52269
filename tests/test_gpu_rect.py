"""Rectangular kernels 1 x k and k x 1 (Section 4.2: Inception-v3's 1 x 7 / 7 x 1 layers) as one-dimensional
Winograd F(m, k) on the GPU, through the C ABI, against the fp64 rectangular direct-convolution oracle."""
import numpy as np
import pytest

from oracle import direct_conv as oc
from paper_2002_12418_b200 import binding as B
from tests.util import assert_close, rel_l2, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available()
    B.lib()
    return torch


def make(N, Cin, Cout, H, W, kh, kw, seed, integer=False):
    rng = np.random.Generator(np.random.PCG64(seed))
    if integer:
        x = rng.integers(-3, 4, size=(N, Cin, H, W)).astype(np.float32)
        w = rng.integers(-3, 4, size=(Cout, Cin, kh, kw)).astype(np.float32)
        b = rng.integers(-3, 4, size=(Cout,)).astype(np.float32)
    else:
        x = np.maximum(rng.standard_normal((N, Cin, H, W), dtype=np.float32), 0)
        w = (rng.standard_normal((Cout, Cin, kh, kw), dtype=np.float32) * np.float32(np.sqrt(2.0 / (Cin * kh * kw)))).astype(np.float32)
        b = (rng.standard_normal((Cout,), dtype=np.float32) * np.float32(0.1)).astype(np.float32)
    return x, w, b


def run_rect(torch, x, w, b, ph, pw, relu=True, **kw):
    N, Cin, H, W = x.shape
    Cout, _, kh, kw_ = w.shape
    plan = B.mnn_conv_plan_rect(N, Cin, Cout, H, W, kh, kw_, ph, pw, B.make_opts(relu=relu, **kw))
    r = B.ConvLayerRunner(N, Cin, Cout, H, W, max(kh, kw_), plan=plan)
    info = r.info
    assert info.rect == (1 if kh == 1 else 2) and info.alpha == info.m + max(kh, kw_) - 1
    assert (info.OH, info.OW) == (H + 2 * ph - kh + 1, W + 2 * pw - kw_ + 1)
    y = r.run(to_dev(torch, x), to_dev(torch, w), to_dev(torch, b))
    torch.cuda.synchronize()
    assert r.device_status() == 0
    out = y.cpu().numpy()
    r.close()
    return out, info


@pytest.mark.parametrize("kh,kw", [(1, 7), (7, 1), (1, 3), (3, 1)])
@pytest.mark.parametrize("C", [128, 192])
@pytest.mark.parametrize("N", [1, 32])
def test_inception_shapes(torch, kh, kw, C, N):
    x, w, b = make(N, C, C, 17, 17, kh, kw, seed=kh * 100 + kw * 10 + C + N)
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    got, info = run_rect(torch, x, w, b, ph, pw)
    ref = oc.direct_conv_rect(x, w, b, ph, pw, True)
    assert_close(got, ref, B.PREC_TF32, "%dx%d C=%d N=%d" % (kh, kw, C, N))


@pytest.mark.parametrize("kh,kw,ph,pw,N,Cin,Cout,H,W", [
    (1, 5, 0, 2, 2, 20, 24, 9, 13), (5, 1, 2, 0, 3, 16, 40, 13, 6), (1, 2, 0, 0, 1, 8, 8, 5, 9), (2, 1, 1, 0, 2, 8, 8, 5, 9),
    (1, 7, 1, 3, 1, 12, 12, 6, 20), (7, 1, 0, 0, 2, 9, 17, 15, 4), (1, 3, 0, 0, 1, 3, 5, 4, 33)])
def test_odd_shapes_and_paddings(torch, kh, kw, ph, pw, N, Cin, Cout, H, W):
    x, w, b = make(N, Cin, Cout, H, W, kh, kw, seed=kh + 3 * kw + H)
    for m in (2, 4):
        if m + max(kh, kw) - 1 > 10:
            continue
        got, _ = run_rect(torch, x, w, b, ph, pw, force_m=m)
        assert_close(got, oc.direct_conv_rect(x, w, b, ph, pw, True), B.PREC_TF32, "m=%d" % m)


@pytest.mark.parametrize("kh,kw", [(1, 3), (3, 1), (1, 7), (7, 1)])
@pytest.mark.parametrize("operand,passes", [(B.OPERAND_TF32, 1), (B.OPERAND_BF16, 3)])
def test_integer_inputs_bit_exact(torch, kh, kw, operand, passes):
    # unit points at alpha = 4 (k = 3, m = 2) and the paper's half-integer points keep every value dyadic
    x, w, b = make(2, 24, 40, 10, 12, kh, kw, seed=5, integer=True)
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    got, _ = run_rect(torch, x, w, b, ph, pw, relu=False, force_m=2, operand=operand, passes=passes, points_id=B.POINTS_PAPER)
    ref = oc.direct_conv_rect(x, w, b, ph, pw, False)
    if max(kh, kw) == 3:
        assert np.array_equal(got.astype(np.float64), ref)
    else:
        # alpha = 8: the matrices hold thirds, so the operands are rounded: near fp32 with the hi + lo split,
        # the single-pass TF32 figure of that tile size otherwise
        assert rel_l2(got, ref) < (1e-4 if passes == 3 else 5e-3)


def test_errors(torch):
    for args in ((1, 8, 8, 8, 8, 3, 3, 1, 1), (1, 8, 8, 8, 8, 1, 1, 0, 0), (1, 8, 8, 8, 8, 1, 4, 0, 0), (1, 8, 8, 2, 2, 7, 1, 0, 0)):
        with pytest.raises(B.MnnError):
            B.mnn_conv_plan_rect(*args, B.make_opts())
    with pytest.raises(B.MnnError):
        B.mnn_conv_plan_rect(1, 8, 8, 8, 8, 1, 7, 0, 3, B.make_opts(force_m=6))
