"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, its generator equals the exact-rational oracle bit for
bit, and the planner's routing invariants hold."""
import os
import re
from fractions import Fraction

import numpy as np
import pytest

from oracle import winograd_exact as wx
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "mnn_conv.h")).read()
    declared = re.findall(r"MNN_API[^;(]*?\b(mnn_\w+)\s*\(", hdr)
    assert len(declared) >= 15 and sorted(declared) == sorted(B.EXPORTED)
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_struct_layouts_match_the_header():
    # sizes follow from the field lists in the header (ints 4 bytes, long long 8)
    import ctypes
    assert ctypes.sizeof(B.ConvOpts) == 16 * 4
    assert ctypes.sizeof(B.ConvInfo) == 16 * 4 + 9 * 8 + 2 * 4 + 16 * 8 + 2 * 4 + 4 * 8 + 2 * 4


@pytest.mark.parametrize("m,k", [(m, k) for m in (1, 2, 3, 4, 6, 8) for k in (1, 2, 3, 5, 7)])
@pytest.mark.parametrize("pid", [1, 2, 3])
def test_generator_matches_exact_oracle_bit_for_bit(m, k, pid):
    if m + k - 1 > 16:
        pytest.skip("alpha > 16")
    At, G, Bt = B.mnn_winograd_matrices(m, k, pid)
    At_o, G_o, Bt_o = wx.matrices_f32(m, k, pid)
    for got, ref in ((At, At_o), (G, G_o), (Bt, Bt_o)):
        got = np.array(got, dtype=np.float32)
        assert got.shape == ref.shape
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


def test_generator_rejects_bad_arguments():
    for args in ((0, 3, 1), (2, 0, 1), (2, 3, 0), (2, 3, 4), (12, 7, 1), (11, 7, 3)):
        with pytest.raises(B.MnnError):
            B.mnn_winograd_matrices(*args)


def test_accuracy_model_orders_the_variants():
    ppm = B.mnn_accuracy_ppm
    for m, k in ((2, 3), (4, 3), (6, 3), (4, 5)):
        for pid in (1, 2, 3):
            if m + k - 1 > 8 and pid == 2:
                continue
            assert ppm(m, k, pid, B.OPERAND_TF32, 1) < ppm(m, k, pid, B.OPERAND_BF16, 1)
            assert ppm(m, k, pid, B.OPERAND_BF16, 3) < ppm(m, k, pid, B.OPERAND_TF32, 1)
            assert ppm(m, k, pid, B.OPERAND_TF32, 3) <= ppm(m, k, pid, B.OPERAND_BF16, 3)
    # larger tiles amplify rounding more
    assert ppm(2, 3, 1, 1, 1) < ppm(4, 3, 1, 1, 1) < ppm(6, 3, 1, 1, 1)
    # deterministic
    assert ppm(4, 3, 1, 1, 1) == ppm(4, 3, 1, 1, 1)


def _plan(layer, **kw):
    o = B.make_opts(groups=layer.groups, relu=layer.relu, **kw)
    p = B.mnn_conv_plan_ex(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad,
                           layer.dilation, o)
    info = B.mnn_conv_plan_query(p)
    B.mnn_conv_destroy(p)
    return info


def test_routing_invariants():
    for cfg in (W.config0(), W.config1(1), W.config1(32), W.config2(1), W.config2(32), W.config3(1), W.config3(64),
                W.config4()):
        for layer in cfg:
            info = _plan(layer)
            assert info.OH == layer.OH and info.OW == layer.OW
            if layer.groups > 1:
                assert info.algo == B.ALGO_DIRECT
            if layer.k == 1:
                assert info.algo != B.ALGO_WINOGRAD        # k = 1 is a matrix product
            if layer.stride > 1 or layer.dilation > 1:
                assert info.algo != B.ALGO_WINOGRAD
            if info.algo == B.ALGO_WINOGRAD:
                assert info.m in (2, 4, 6) and info.alpha == info.m + layer.k - 1
                assert info.predicted_error_ppm <= 700       # the accuracy gate of class TF32
                assert info.n_chunks * info.chunk_images >= layer.N
            chosen = info.chosen_candidate
            costs = list(info.cost_ps)
            assert costs[chosen] == min(costs) and costs.index(min(costs)) == chosen    # first minimum wins


def test_inadmissible_variants_are_never_chosen():
    layer = W.config1(32)[0]
    info = _plan(layer)
    costs = list(info.cost_ps)
    # single-pass TF32 with m = 4 or 6 and every single-pass BF16 variant miss 1e-3
    for idx in (4, 5, 9, 10, 11):
        assert costs[idx] == B.COST_INADMISSIBLE
    info_b = _plan(layer, precision=B.PREC_BF16)
    assert list(info_b.cost_ps)[4] != B.COST_INADMISSIBLE      # tf32 m=4 passes the 1e-2 class


def test_cost_is_monotone_in_batch():
    prev = None
    for n in (1, 2, 4, 8, 16, 32, 64):
        layer = W.config1(1)[1].with_batch(n)
        costs = list(_plan(layer).cost_ps)
        if prev is not None:
            for a, b in zip(prev, costs):
                if a != B.COST_INADMISSIBLE:
                    assert b >= a
        prev = costs


def test_forced_options_and_errors():
    layer = W.config0()[0]
    info = _plan(layer, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=B.OPERAND_TF32, passes=1, points_id=1)
    assert (info.algo, info.m, info.operand, info.passes, info.points_id) == (B.ALGO_WINOGRAD, 4, B.OPERAND_TF32, 1, 1)
    assert info.workspace_bytes > 0 and info.u_offset % 1024 == 0 and info.v_offset % 1024 == 0 and info.m_offset % 1024 == 0
    with pytest.raises(B.MnnError):
        B.mnn_conv_plan_ex(1, 32, 32, 28, 28, 3, 2, 1, 1, B.make_opts(force_algo=B.ALGO_WINOGRAD))   # stride 2
    with pytest.raises(B.MnnError):
        B.mnn_conv_plan(0, 32, 32, 28, 28, 3, 1, 1, 1)
    with pytest.raises(B.MnnError):
        B.mnn_conv_plan(1, 32, 32, 2, 2, 5, 1, 0, 1)            # kernel larger than the input
    with pytest.raises(B.MnnError):
        B.mnn_conv_plan_ex(1, 6, 6, 8, 8, 3, 1, 1, 1, B.make_opts(groups=4))
    assert "groups" in B.mnn_last_error()


def test_gemm_left_operand_option():
    def plan(N, Cin, Cout, H, W_, k, stride, pad, **kw):
        h = B.mnn_conv_plan_ex(N, Cin, Cout, H, W_, k, stride, pad, 1, B.make_opts(relu=1, **kw))
        info = B.mnn_conv_plan_query(h)
        B.mnn_conv_destroy(h)
        return info
    gemm = dict(force_algo=B.ALGO_GEMM, operand=B.OPERAND_TF32, passes=1)
    # x itself: one launch, no patch matrix in the workspace, a smaller workspace than with patches
    ix = plan(4, 64, 96, 14, 14, 1, 1, 0, gemm_lhs=B.GEMM_LHS_X, **gemm)
    ip = plan(4, 64, 96, 14, 14, 1, 1, 0, gemm_lhs=B.GEMM_LHS_PATCHES, **gemm)
    assert (ix.gemm_lhs, ix.launches_per_run, ix.v_bytes) == (B.GEMM_LHS_X, 1, 0)
    assert (ip.gemm_lhs, ip.launches_per_run) == (B.GEMM_LHS_PATCHES, 2) and ip.v_bytes >= 4 * 4 * 196 * 64
    assert ix.workspace_bytes < ip.workspace_bytes
    assert ix.predicted_error_ppm >= ip.predicted_error_ppm          # truncation instead of rounding
    # left to the planner the choice is one of the two and is reported; other schemes report 0
    ia = plan(4, 64, 96, 14, 14, 1, 1, 0, **gemm)
    assert ia.gemm_lhs in (B.GEMM_LHS_X, B.GEMM_LHS_PATCHES)
    assert plan(1, 32, 32, 28, 28, 3, 1, 1, force_algo=B.ALGO_WINOGRAD).gemm_lhs == 0
    # where x cannot be the operand, asking for it fails the plan; patches still plan
    for shape in [(1, 64, 64, 14, 14, 3, 1, 1), (1, 64, 64, 14, 14, 1, 2, 0), (1, 64, 64, 7, 7, 1, 1, 0),
                  (1, 64, 64, 4, 4, 1, 1, 0), (1, 64, 64, 14, 14, 1, 1, 1)]:
        with pytest.raises(B.MnnError):
            plan(*shape, gemm_lhs=B.GEMM_LHS_X, **gemm)
        assert plan(*shape, gemm_lhs=B.GEMM_LHS_PATCHES, **gemm).gemm_lhs == B.GEMM_LHS_PATCHES
    with pytest.raises(B.MnnError):                                   # BF16 operands need the rounded copy
        plan(4, 64, 96, 14, 14, 1, 1, 0, force_algo=B.ALGO_GEMM, operand=B.OPERAND_BF16, precision=B.PREC_BF16,
             gemm_lhs=B.GEMM_LHS_X)


def test_calibration_record_round_trip_changes_the_plan():
    base = B.mnn_get_calibration()
    try:
        layer = W.config1(32)[0]
        before = list(_plan(layer).cost_ps)
        slow_tensor = list(base)
        slow_tensor[2] *= 100
        slow_tensor[3] *= 100
        B.mnn_set_calibration(slow_tensor)
        assert B.mnn_get_calibration() == slow_tensor
        after = list(_plan(layer).cost_ps)
        assert after != before and after[0] == before[0]        # the direct kernel does not use tensor cores
        with pytest.raises(B.MnnError):
            B.mnn_set_calibration([0] * 16)
    finally:
        B.mnn_set_calibration(base)
