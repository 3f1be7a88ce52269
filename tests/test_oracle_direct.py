"""Pins for the fp64 direct-convolution oracle: hand-worked values, closed
forms, invariants and an independently ordered evaluation on tiny shapes."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import direct_conv as oc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def shift_and_add(x, w, bias, stride, pad, dil, groups, relu):
    """Second evaluation with a different loop order: for every tap (a, b) add a
    strided slice of the zero-padded image times the tap's channel matrix."""
    x = x.astype(np.float64)
    w = w.astype(np.float64)
    N, Cin, H, W = x.shape
    Cout, cpg, k, _ = w.shape
    OH = (H + 2 * pad - dil * (k - 1) - 1) // stride + 1
    OW = (W + 2 * pad - dil * (k - 1) - 1) // stride + 1
    xp = np.zeros((N, Cin, H + 2 * pad, W + 2 * pad))
    xp[:, :, pad:pad + H, pad:pad + W] = x
    y = np.zeros((N, Cout, OH, OW))
    opg = Cout // groups
    for b in range(k):
        for a in range(k):
            sl = xp[:, :, a * dil: a * dil + (OH - 1) * stride + 1: stride,
                    b * dil: b * dil + (OW - 1) * stride + 1: stride]
            for g in range(groups):
                y[:, g * opg:(g + 1) * opg] += np.einsum("oc,nchw->nohw", w[g * opg:(g + 1) * opg, :, a, b],
                                                         sl[:, g * cpg:(g + 1) * cpg])
    if bias is not None:
        y += bias.astype(np.float64)[None, :, None, None]
    if relu:
        y = np.maximum(y, 0)
    return y


def test_hand_worked_cases():
    with open(os.path.join(GOLDEN, "hand_conv_cases.json")) as f:
        cases = json.load(f)["cases"]
    assert len(cases) == 3
    for c in cases:
        x = np.array(c["x"], dtype=np.float32).reshape(c["x_shape"])
        w = np.array(c["w"], dtype=np.float32).reshape(c["w_shape"])
        y = oc.direct_conv(x, w, None, c["stride"], c["pad"], c["dil"], c["groups"], False)
        assert list(y.shape) == c["y_shape"], c["name"]
        assert y.ravel().tolist() == [float(v) for v in c["y"]], c["name"]


@pytest.mark.parametrize("k,stride,pad,dil", [(k, s, p, d) for k in (1, 2, 3) for s in (1, 2, 3)
                                               for p in (0, 1, 2) for d in (1, 2)])
def test_against_reordered_evaluation(k, stride, pad, dil):
    rng = np.random.default_rng(100 * k + 10 * stride + pad + 7 * dil)
    for (N, Cin, Cout, H, W, groups) in [(2, 3, 2, 7, 6, 1), (1, 4, 6, 5, 7, 2), (2, 3, 3, 6, 5, 3)]:
        if H + 2 * pad < dil * (k - 1) + 1 or W + 2 * pad < dil * (k - 1) + 1:
            continue
        x = rng.standard_normal((N, Cin, H, W)).astype(np.float32)
        w = rng.standard_normal((Cout, Cin // groups, k, k)).astype(np.float32)
        b = rng.standard_normal(Cout).astype(np.float32)
        for relu in (False, True):
            got = oc.direct_conv(x, w, b, stride, pad, dil, groups, relu)
            ref = shift_and_add(x, w, b, stride, pad, dil, groups, relu)
            assert got.shape == ref.shape
            np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_delta_kernel_returns_input():
    rng = np.random.default_rng(3)
    for k in (1, 3, 5, 7):
        C = 4
        x = rng.standard_normal((2, C, 9, 8)).astype(np.float32)
        w = np.zeros((C, C, k, k), dtype=np.float32)
        for c in range(C):
            w[c, c, k // 2, k // 2] = 1.0
        y = oc.direct_conv(x, w, None, 1, k // 2, 1, 1, False)
        assert np.array_equal(y, x.astype(np.float64))


def test_off_centre_delta_shifts_the_right_way():
    # tap (a, b) = (0, 2) of a 3x3 kernel with pad 1: y[oh, ow] = x[oh - 1, ow + 1]
    x = np.arange(30, dtype=np.float32).reshape(1, 1, 5, 6)
    w = np.zeros((1, 1, 3, 3), dtype=np.float32)
    w[0, 0, 0, 2] = 1.0
    y = oc.direct_conv(x, w, None, 1, 1, 1, 1, False)[0, 0]
    expect = np.zeros((5, 6))
    expect[1:, :-1] = x[0, 0, :-1, 1:]
    assert np.array_equal(y, expect)


def test_linearity_in_x_and_w():
    rng = np.random.default_rng(5)
    # dyadic values keep every fp32 combination exact, so linearity is exact to fp64 rounding
    x1 = (rng.integers(-64, 64, (2, 3, 8, 8)) / 16).astype(np.float32)
    x2 = (rng.integers(-64, 64, (2, 3, 8, 8)) / 16).astype(np.float32)
    w1 = (rng.integers(-64, 64, (4, 3, 3, 3)) / 16).astype(np.float32)
    w2 = (rng.integers(-64, 64, (4, 3, 3, 3)) / 16).astype(np.float32)
    f = lambda x, w: oc.direct_conv(x, w, None, 2, 1, 1, 1, False)
    np.testing.assert_allclose(f(2 * x1 + x2, w1), 2 * f(x1, w1) + f(x2, w1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(f(x1, w1 - 3 * w2), f(x1, w1) - 3 * f(x1, w2), rtol=0, atol=1e-12)


def test_k1_is_a_matrix_product():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((3, 5, 4, 7)).astype(np.float32)
    w = rng.standard_normal((6, 5, 1, 1)).astype(np.float32)
    y = oc.direct_conv(x, w, None, 1, 0, 1, 1, False)
    ref = np.matmul(w[:, :, 0, 0].astype(np.float64), x.astype(np.float64).reshape(3, 5, 28)).reshape(3, 6, 4, 7)
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)
    # stride 2 sub-samples the input first
    y2 = oc.direct_conv(x, w, None, 2, 0, 1, 1, False)
    np.testing.assert_allclose(y2, ref[:, :, ::2, ::2], rtol=0, atol=1e-12)


def test_box_sum_closed_form():
    # all-ones image and kernel: the output counts the taps that land inside the image
    for k, pad, dil in itertools.product((3, 5), (0, 1, 2), (1, 2)):
        H, W, C = 9, 11, 3
        x = np.ones((1, C, H, W), dtype=np.float32)
        w = np.ones((2, C, k, k), dtype=np.float32)
        y = oc.direct_conv(x, w, None, 1, pad, dil, 1, False)
        OH, OW = y.shape[2:]
        for oh in range(OH):
            rows = sum(0 <= oh - pad + a * dil < H for a in range(k))
            for ow in range(OW):
                cols = sum(0 <= ow - pad + b * dil < W for b in range(k))
                assert y[0, 0, oh, ow] == C * rows * cols == y[0, 1, oh, ow]


def test_bias_and_relu_order():
    x = np.ones((1, 1, 2, 2), dtype=np.float32)
    w = -np.ones((2, 1, 1, 1), dtype=np.float32)
    b = np.array([0.5, 2.0], dtype=np.float32)
    y = oc.direct_conv(x, w, b, 1, 0, 1, 1, True)
    assert np.array_equal(y[0, 0], np.zeros((2, 2)))          # relu(-1 + 0.5) = 0
    assert np.array_equal(y[0, 1], np.ones((2, 2)))           # relu(-1 + 2) = 1


def test_depthwise_is_per_channel():
    rng = np.random.default_rng(8)
    C = 5
    x = rng.standard_normal((2, C, 6, 6)).astype(np.float32)
    w = rng.standard_normal((C, 1, 3, 3)).astype(np.float32)
    y = oc.direct_conv(x, w, None, 1, 1, 1, C, False)
    for c in range(C):
        yc = oc.direct_conv(x[:, c:c + 1], w[c:c + 1], None, 1, 1, 1, 1, False)
        assert np.array_equal(y[:, c:c + 1], yc)


def test_partial_entry_points_agree_with_full():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((4, 3, 7, 7)).astype(np.float32)
    w = rng.standard_normal((5, 3, 3, 3)).astype(np.float32)
    b = rng.standard_normal(5).astype(np.float32)
    full = oc.direct_conv(x, w, b, 2, 1, 1, 1, True)
    some = oc.direct_conv_images(x, w, b, [3, 0], 2, 1, 1, 1, True)
    assert np.array_equal(some[0], full[3]) and np.array_equal(some[1], full[0])
    idx = rng.integers(0, full.size, 50)
    assert np.array_equal(oc.direct_conv_at(x, w, b, idx, 2, 1, 1, 1, True), full.ravel()[idx])


def test_rejects_bad_arguments():
    x = np.zeros((1, 3, 4, 4), dtype=np.float32)
    w = np.zeros((4, 3, 3, 3), dtype=np.float32)
    with pytest.raises(ValueError):
        oc.direct_conv(x, w, None, 1, 0, 1, 2, False)       # 3 channels, 2 groups
    with pytest.raises(ValueError):
        oc.direct_conv(x, w, None, 0, 0, 1, 1, False)       # stride 0


# ---------------------------------------------------------------------------
# Rectangular kernels (Section 4.2: the 1 x 7 / 7 x 1 convolutions of Inception-v3).
# ---------------------------------------------------------------------------
def test_rect_hand_worked_cases():
    import json
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "hand_rect_cases.json")
    for case in json.load(open(path))["cases"]:
        x = np.array(case["x"], dtype=np.float32)
        w = np.array(case["w"], dtype=np.float32)
        b = np.array(case["bias"], dtype=np.float32)
        y = oc.direct_conv_rect(x, w, b, case["pad_h"], case["pad_w"], case["relu"])
        assert np.array_equal(y, np.array(case["y"], dtype=np.float64)), case["name"]


def _rect_other_order(x, w, b, ph, pw, relu):
    """A second evaluation: one shifted, zero-padded copy of x per kernel tap, accumulated tap by tap."""
    N, Cin, H, W = x.shape
    Cout, _, kh, kw = w.shape
    OH, OW = H + 2 * ph - kh + 1, W + 2 * pw - kw + 1
    xp = np.zeros((N, Cin, H + 2 * ph, W + 2 * pw))
    xp[:, :, ph:ph + H, pw:pw + W] = x
    y = np.zeros((N, Cout, OH, OW))
    for a in range(kh):
        for c in range(kw):
            y += np.einsum("oc,nchw->nohw", w[:, :, a, c].astype(np.float64), xp[:, :, a:a + OH, c:c + OW])
    y += b.astype(np.float64)[None, :, None, None]
    return np.maximum(y, 0) if relu else y


@pytest.mark.parametrize("kh,kw,ph,pw", [(1, 3, 0, 1), (3, 1, 1, 0), (1, 7, 0, 3), (7, 1, 3, 0), (1, 5, 1, 0), (2, 3, 1, 2),
                                         (3, 3, 1, 1), (1, 1, 0, 0)])
def test_rect_against_a_second_evaluation_order(kh, kw, ph, pw):
    rng = np.random.default_rng(kh * 10 + kw)
    x = rng.standard_normal((2, 3, 6, 9)).astype(np.float32)
    w = rng.standard_normal((4, 3, kh, kw)).astype(np.float32)
    b = rng.standard_normal(4).astype(np.float32)
    for relu in (False, True):
        got = oc.direct_conv_rect(x, w, b, ph, pw, relu)
        assert np.allclose(got, _rect_other_order(x, w, b, ph, pw, relu), rtol=0, atol=1e-12)


def test_rect_reduces_to_the_square_definition_and_transposes():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((2, 3, 7, 8)).astype(np.float32)
    w = rng.standard_normal((5, 3, 3, 3)).astype(np.float32)
    b = rng.standard_normal(5).astype(np.float32)
    assert np.array_equal(oc.direct_conv_rect(x, w, b, 1, 1, True), oc.direct_conv(x, w, b, 1, 1, 1, 1, True))
    # a 1 x k kernel on x equals the k x 1 kernel on the transposed image, transposed back
    w17 = rng.standard_normal((5, 3, 1, 7)).astype(np.float32)
    a = oc.direct_conv_rect(x, w17, b, 0, 3)
    t = oc.direct_conv_rect(x.transpose(0, 1, 3, 2), w17.transpose(0, 1, 3, 2), b, 3, 0)
    assert np.array_equal(a, t.transpose(0, 1, 3, 2))
    # an off-centre delta tap shifts the image (catches a flipped kernel)
    d = np.zeros((1, 1, 1, 3), dtype=np.float32)
    d[0, 0, 0, 2] = 1
    img = rng.standard_normal((1, 1, 2, 6)).astype(np.float32)
    y = oc.direct_conv_rect(img, d, None, 0, 1)
    assert np.array_equal(y[0, 0, :, :5], img[0, 0, :, 1:].astype(np.float64)) and not y[0, 0, :, 5].any()
