"""Pins for the exact-rational Winograd oracle (Eq. 6, Eq. 8)."""
import json
import os
import random
from fractions import Fraction

import numpy as np
import pytest

from oracle import direct_conv as oc
from oracle import winograd_exact as wx

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MK = [(m, k) for m in (1, 2, 3, 4, 6) for k in (1, 2, 3, 5, 7)]
POINT_SETS = (wx.POINTS_PAPER, wx.POINTS_UNIT, wx.POINTS_MIXED)


def test_point_sets():
    h = Fraction(1, 2)
    assert wx.interpolation_points(6, wx.POINTS_PAPER) == [0, h, -h, 1, -1]
    assert wx.interpolation_points(4, wx.POINTS_UNIT) == [0, 1, -1]
    assert wx.interpolation_points(8, wx.POINTS_MIXED) == [0, 1, -1, h, -h, 2, -2]
    # odd alpha (even k): the asymmetric set 0, f, -f, 2f
    assert wx.interpolation_points(5, wx.POINTS_PAPER) == [0, h, -h, 1]
    assert wx.interpolation_points(1, wx.POINTS_PAPER) == []


def test_last_row_of_Bt_is_the_generator_polynomial():
    # Eq. 8 for alpha = 6, f = 1/2: x (x-1/2)(x+1/2)(x-1)(x+1) = x^5 - 5/4 x^3 + 1/4 x
    _, _, Bt = wx.generate(4, 3, wx.POINTS_PAPER)
    assert Bt[-1] == [0, Fraction(1, 4), 0, Fraction(-5, 4), 0, 1]


@pytest.mark.parametrize("m,k", MK)
@pytest.mark.parametrize("pid", POINT_SETS)
def test_1d_identity_is_exact(m, k, pid):
    rnd = random.Random(1000 * m + 10 * k + pid)
    alpha = m + k - 1
    for _ in range(5):
        d = [rnd.randint(-9, 9) for _ in range(alpha)]
        g = [rnd.randint(-9, 9) for _ in range(k)]
        y = wx.winograd_1d_exact(d, g, m, pid)
        ref = [sum(d[j + i] * g[i] for i in range(k)) for j in range(m)]
        assert y == ref


@pytest.mark.parametrize("m,k", [(2, 3), (4, 3), (6, 3), (4, 5), (2, 7), (3, 2)])
def test_2d_tile_identity_is_exact(m, k):
    rnd = random.Random(m * 31 + k)
    alpha = m + k - 1
    C = 3
    X = [[[rnd.randint(-5, 5) for _ in range(alpha)] for _ in range(alpha)] for _ in range(C)]
    Wk = [[[rnd.randint(-5, 5) for _ in range(k)] for _ in range(k)] for _ in range(C)]
    Y = wx.winograd_2d_tile_exact(X, Wk, m)
    for a in range(m):
        for b in range(m):
            ref = sum(X[c][a + i][b + j] * Wk[c][i][j] for c in range(C) for i in range(k) for j in range(k))
            assert Y[a][b] == ref


def test_m1_degenerates_to_the_definition():
    # alpha = k: every matrix is square and the "transform" is a change of basis of the dot product
    A, G, Bt = wx.generate(1, 3, wx.POINTS_PAPER)
    assert len(A) == 3 and len(A[0]) == 1 and all(r == [1] for r in A[:-1]) and A[-1] == [1]
    d, g = [3, -1, 4], [2, 7, -5]
    assert wx.winograd_1d_exact(d, g, 1) == [3 * 2 - 7 - 20]


def test_unit_points_reproduce_the_textbook_f23():
    with open(os.path.join(GOLDEN, "lavin_f23.json")) as f:
        gold = json.load(f)
    A, G, Bt = wx.generate(2, 3, wx.POINTS_UNIT)

    def triples(A_rows, G_rows, Bt_rows):
        out = set()
        for a, g, b in zip(A_rows, G_rows, Bt_rows):
            t = tuple(Fraction(x) * Fraction(y) * Fraction(z) for x in a for y in g for z in b)
            out.add(t)
        return out

    gold_A = [list(c) for c in zip(*[[Fraction(v) for v in r] for r in gold["At"]])]
    gold_G = [[Fraction(v) for v in r] for r in gold["G"]]
    gold_Bt = [[Fraction(v) for v in r] for r in gold["Bt"]]
    assert triples(A, G, Bt) == triples(gold_A, gold_G, gold_Bt)


@pytest.mark.parametrize("m,k,pad,H,W", [(2, 3, 1, 5, 7), (4, 3, 1, 7, 6), (6, 3, 0, 9, 8), (2, 5, 2, 6, 6),
                                         (4, 2, 0, 6, 5)])
def test_whole_convolution_exact_with_ragged_edges(m, k, pad, H, W):
    rng = np.random.default_rng(m * 100 + k)
    x = rng.integers(-3, 4, (2, 2, H, W))
    w = rng.integers(-3, 4, (3, 2, k, k))
    got = wx.winograd_conv_exact(x, w, m, pad)
    ref = oc.direct_conv(x.astype(np.float32), w.astype(np.float32), None, 1, pad, 1, 1, False)
    got_arr = np.array([[[[float(v) for v in row] for row in ch] for ch in img] for img in got])
    assert got_arr.shape == ref.shape
    assert np.array_equal(got_arr, ref)           # integers: both sides exact


@pytest.mark.parametrize("m,k,pid", [(2, 3, 1), (2, 3, 2), (4, 3, 1), (6, 3, 1), (6, 3, 3), (4, 5, 1), (2, 7, 1)])
def test_fp64_stage_chain_matches_direct(m, k, pid):
    rng = np.random.default_rng(m + 10 * k)
    pad = k // 2
    x = rng.standard_normal((2, 5, 11, 9)).astype(np.float32)
    w = rng.standard_normal((4, 5, k, k)).astype(np.float32)
    b = rng.standard_normal(4).astype(np.float32)
    y = wx.winograd_conv_f64(x, w, m, pad, b, True, pid)
    ref = oc.direct_conv(x, w, b, 1, pad, 1, 1, True)
    err = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    assert err < 1e-11, err


def test_fp32_rounding_of_matrices():
    At, G, Bt = wx.matrices_f32(4, 3, wx.POINTS_PAPER)
    A_ex, G_ex, Bt_ex = wx.generate(4, 3, wx.POINTS_PAPER)
    for i in range(6):
        for j in range(3):
            v = G_ex[i][j]
            got = Fraction(float(G[i, j]))
            # within half an ulp of the exact value
            assert abs(got - v) <= abs(v) * Fraction(1, 2 ** 24)
    assert At.shape == (4, 6) and Bt.shape == (6, 6) and At.dtype == np.float32
    # entries with short binary expansions are exact
    assert Fraction(float(Bt[5, 3])) == Fraction(-5, 4)


def test_round_to_mantissa():
    a = np.array([1.0, 1.0 + 2 ** -11, 1.0 + 3 * 2 ** -11, 1.0 + 2 ** -10, -3.1415927], dtype=np.float32)
    r = wx.round_to_mantissa(a, 10)
    # ties go to the even 10-bit mantissa
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -9 and r[3] == 1.0 + 2 ** -10
    assert abs(r[4] + 3.1415927) <= 2 ** -10
    b = wx.round_to_mantissa(np.array([1.0 + 2 ** -8 + 2 ** -9], dtype=np.float32), 7)
    assert b[0] == 1.0 + 2 ** -7
