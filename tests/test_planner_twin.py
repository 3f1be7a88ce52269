"""The planner (Section 3.2, Eq. 1-5) against its Python-integer twin, and the twin against what
arithmetic fixes.  No GPU: planning is host work.

* every layer of configs 0-4, both batch sizes, both accuracy classes, two calibration records
  (built-in and a perturbed one): every cost_ps[i] and every field of the decision bit-equal;
* two fresh processes given the same frozen record return byte-identical mnn_conv_info;
* the accuracy gate's integers (ppm) reproduced by an fp64 restatement of the model on the exact
  rational generator's matrices;
* the twin itself: hand-computed costs, the tie-break, saturation, Eq. 2 on a worked example.
"""
import functools
import json
import os
import subprocess
import sys

import pytest

from oracle import planner_twin as T
from oracle import winograd_exact as wx
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@functools.lru_cache(maxsize=None)
def ppm_table():
    """The accuracy model's integers, read through the ABI, as the twin's input table."""
    t = {}
    for k in (1, 2, 3, 5, 7):
        for operand in (B.OPERAND_TF32, B.OPERAND_BF16):
            for passes in (1, 3):
                t[(1, k, 0, operand, passes)] = B.mnn_accuracy_ppm(1, k, 0, operand, passes)
                if k == 1:
                    continue
                for m in (2, 4, 6):
                    if m + k - 1 > 12:
                        continue
                    for pid in (1, 2, 3):
                        try:
                            t[(m, k, pid, operand, passes)] = B.mnn_accuracy_ppm(m, k, pid, operand, passes)
                        except B.MnnError:
                            pass
    return t


def all_layers():
    out = []
    for cfg in (W.config0(), W.config1(1), W.config1(32), W.config2(1), W.config2(32), W.config3(1), W.config3(64),
                W.config4(64)):
        out += cfg
    return out


def twin_layer(l):
    return T.Layer(l.N, l.Cin, l.Cout, l.H, l.W, l.k, l.stride, l.pad, l.dilation, l.groups)


def compare(l, opts_kw, twin_kw, cal):
    o = B.make_opts(groups=l.groups, relu=l.relu, **opts_kw)
    plan = B.mnn_conv_plan_ex(l.N, l.Cin, l.Cout, l.H, l.W, l.k, l.stride, l.pad, l.dilation, o)
    info = B.mnn_conv_plan_query(plan)
    B.mnn_conv_destroy(plan)
    ch = T.plan(twin_layer(l), T.Options(**twin_kw), cal, ppm_table())
    what = "%s %s" % (l.name, opts_kw)
    assert list(info.cost_ps) == ch.cost_ps, what
    got = (info.chosen_candidate, info.algo, info.m, info.operand, info.passes, info.points_id, info.gemm_lhs,
           info.chunk_images, info.n_chunks, info.fused, info.predicted_error_ppm)
    want = (ch.chosen, ch.algo, ch.m, ch.operand, ch.passes, ch.points_id, ch.gemm_lhs, ch.chunk_images, ch.n_chunks,
            ch.fused, ch.error_ppm)
    assert got == want, what
    n_hat, counts = T.paper_choice(twin_layer(l))
    assert (info.paper_n_hat, list(info.paper_mul)) == (n_hat, counts), what
    return info


@pytest.fixture()
def restore_calibration():
    B.lib()
    before = B.mnn_get_calibration()
    yield before
    B.mnn_set_calibration(before)


PERTURBED = [211000, 61000, 2500, 900, 35000, 5100000, 40 << 20, 132, 480000, 45000, 15000, 900000, 2500000, 90000000, 0, 0]


@pytest.mark.parametrize("record", ["builtin", "perturbed"])
def test_every_config_layer_matches_the_twin(restore_calibration, record):
    cal = list(restore_calibration) if record == "builtin" else PERTURBED
    B.mnn_set_calibration(cal)
    assert B.mnn_get_calibration() == cal
    n = 0
    for l in all_layers():
        for prec in (B.PREC_TF32, B.PREC_BF16):
            compare(l, dict(precision=prec), dict(precision=prec), cal)
            n += 1
    assert n >= 200


def test_forced_options_match_the_twin(restore_calibration):
    cal = list(restore_calibration)
    l = W.config1(32)[1]
    cases = [
        (dict(force_algo=B.ALGO_WINOGRAD), dict(force_algo=T.ALGO_WINOGRAD)),
        (dict(force_algo=B.ALGO_GEMM), dict(force_algo=T.ALGO_GEMM)),
        (dict(force_algo=B.ALGO_DIRECT), dict(force_algo=T.ALGO_DIRECT)),
        (dict(force_m=4), dict(force_m=4)),
        (dict(operand=B.OPERAND_BF16), dict(operand=T.OPERAND_BF16)),
        (dict(passes=3), dict(passes=3)),
        (dict(points_id=1), dict(points_id=1)),
        (dict(fused=B.FUSED_NEVER), dict(fused=1)),
        (dict(fused=B.FUSED_ONLY), dict(fused=2)),
        (dict(force_m=6, operand=B.OPERAND_TF32, passes=1), dict(force_m=6, operand=T.OPERAND_TF32, passes=1)),
    ]
    for okw, tkw in cases:
        compare(l, okw, tkw, cal)
    pw = W.config3(64)[2]
    for lhs in (B.GEMM_LHS_PATCHES, B.GEMM_LHS_X, B.GEMM_LHS_IMPLICIT):
        compare(pw, dict(gemm_lhs=lhs), dict(gemm_lhs=lhs), cal)
    s2 = W.config2(32)[5]                                   # 3x3 stride 2: patches or the implicit gather
    for lhs in (B.GEMM_LHS_PATCHES, B.GEMM_LHS_IMPLICIT):
        compare(s2, dict(force_algo=B.ALGO_GEMM, gemm_lhs=lhs), dict(force_algo=T.ALGO_GEMM, gemm_lhs=lhs), cal)
    fast = list(cal)
    fast[13] = 1000                                         # a gather that costs nothing: the planner takes it by itself
    B.mnn_set_calibration(fast)
    info = compare(s2, dict(force_algo=B.ALGO_GEMM), dict(force_algo=T.ALGO_GEMM), fast)
    assert info.gemm_lhs == B.GEMM_LHS_IMPLICIT


def test_fused_candidate_disappears_without_its_constants(restore_calibration):
    cal = list(restore_calibration)
    cal[10] = 0
    B.mnn_set_calibration(cal)
    info = compare(W.config1(32)[0], {}, {}, cal)
    assert info.cost_ps[15] == B.COST_INADMISSIBLE


def test_very_large_layers_saturate_instead_of_wrapping(restore_calibration):
    cal = list(restore_calibration)
    # just under the 2^40-element limit of the ABI: attosecond products pass 2^64
    big = W.ConvLayer("huge", 4096, 1024, 1024, 500, 500, 3, 1, 1, seed=1)
    info = compare(big, {}, {}, cal)
    finite = [c for c in info.cost_ps if c != B.COST_INADMISSIBLE]
    small = W.ConvLayer("small", 1, 1024, 1024, 500, 500, 3, 1, 1, seed=1)
    info_small = compare(small, {}, {}, cal)
    for a, b in zip(info.cost_ps, info_small.cost_ps):
        if a != B.COST_INADMISSIBLE:
            assert a > b                                   # 4096 images never cost less than one
    assert finite


def test_two_fresh_processes_return_identical_bytes():
    code = r"""
import ctypes, sys, json
sys.path.insert(0, %r)
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
B.mnn_set_calibration(%r)
out = []
for cfg in (W.config1(32), W.config3(64), W.config4(64)):
    for l in cfg:
        for prec in (0, 1):
            p = B.mnn_conv_plan_ex(l.N, l.Cin, l.Cout, l.H, l.W, l.k, l.stride, l.pad, l.dilation,
                                   B.make_opts(groups=l.groups, relu=l.relu, precision=prec))
            out.append(bytes(B.mnn_conv_plan_query(p)).hex())
            B.mnn_conv_destroy(p)
print(json.dumps(out))
""" % (ROOT, PERTURBED)
    runs = [subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, check=True).stdout for _ in range(2)]
    a, b = json.loads(runs[0]), json.loads(runs[1])
    assert len(a) == 2 * (4 + 27 + 4) and a == b


# ---------------------------------------------------------------------------
# The accuracy gate's integers.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("m,k", [(1, 1), (1, 3), (1, 7), (2, 3), (4, 3), (6, 3), (2, 5), (4, 5), (2, 7), (4, 7), (6, 7)])
def test_accuracy_model_matches_its_fp64_restatement(m, k):
    B.lib()
    for operand in (B.OPERAND_TF32, B.OPERAND_BF16):
        for passes in (1, 3):
            for pid in ((0,) if m == 1 else (1, 2, 3)):
                try:
                    lib = B.mnn_accuracy_ppm(m, k, pid, operand, passes)
                except B.MnnError:
                    continue
                twin = T.accuracy_ppm(m, k, pid, operand, passes, generate=wx.generate)
                # the two sum in different orders: equal up to the last unit of a value that is rounded up
                assert abs(lib - twin) <= max(1, lib // 10 ** 9), (m, k, pid, operand, passes, lib, twin)


def test_accuracy_gate_separates_what_the_tolerances_separate():
    t = ppm_table()
    # one TF32 pass meets 1e-3 (with the 0.7 margin) only at m = 2; three passes always do for alpha <= 10
    assert min(t[(2, 3, p, B.OPERAND_TF32, 1)] for p in (1, 2, 3)) <= 700
    assert min(t[(4, 3, p, B.OPERAND_TF32, 1)] for p in (1, 2, 3)) > 700
    assert min(t[(4, 3, p, B.OPERAND_BF16, 3)] for p in (1, 2, 3)) <= 700
    assert min(t[(6, 3, p, B.OPERAND_BF16, 1)] for p in (1, 2, 3)) > 7000


# ---------------------------------------------------------------------------
# The twin against arithmetic done by hand.
# ---------------------------------------------------------------------------
CAL = [100000, 50000, 2000, 1000, 20000, 3000000, 64 << 20, 100, 500000, 50000, 10000, 1000000, 2000000, 0, 0, 0]


def test_kernel_cost_is_the_largest_bound_plus_the_launch_term():
    assert T.kernel_ps(CAL) == 3000000
    assert T.kernel_ps(CAL, mem_as=7 * 10 ** 12) == 7000000 + 3000000
    assert T.kernel_ps(CAL, mem_as=7 * 10 ** 12, tensor_as=9 * 10 ** 12, alu_as=8 * 10 ** 12) == 9000000 + 3000000
    assert T.kernel_ps(CAL, mem_as=1999999) == 1 + 3000000           # truncating division
    assert T.kernel_ps(CAL, mem_as=2 ** 200) == T.SATURATED


def test_direct_cost_by_hand():
    # 1 image, 2 -> 3 channels, 4 x 4, k = 3, pad 1: 4 x 4 outputs
    L = T.Layer(1, 2, 3, 4, 4, 3, 1, 1)
    traffic = 4 * (2 * 16 + 3 * 16 + 3 * 2 * 9)            # 536 bytes
    flops = 2 * 3 * 2 * 16 * 9                              # 1728
    # two input channels: twice the few-channel rate constant c[9] (c[9] itself is the 3 -> Cout 3x3 stride-2 kernel's)
    assert T.direct_cost(L, CAL) == max(traffic * 100000, flops * 2 * 50000) // 10 ** 6 + 3000000
    Ls = T.Layer(2, 3, 32, 8, 8, 3, 2, 1)                   # that kernel's shape: 4 x 4 outputs
    tr = 4 * (2 * 3 * 64 + 2 * 32 * 16 + 32 * 27)
    fl = 2 * 2 * 32 * 3 * 16 * 9
    assert T.direct_cost(Ls, CAL) == max(tr * 100000, fl * 50000) // 10 ** 6 + 3000000
    assert T.direct_cost(T.Layer(2, 3, 32, 8, 8, 3, 1, 1), CAL) > 0 and \
        T.direct_cost(T.Layer(2, 3, 32, 8, 6, 3, 2, 1), CAL) == \
        max(4 * (2 * 3 * 48 + 2 * 32 * 12 + 32 * 27) * 100000, 2 * 2 * 32 * 3 * 12 * 9 * 2 * 50000) // 10 ** 6 + 3000000
    L8 = T.Layer(1, 8, 3, 4, 4, 3, 1, 1)
    assert T.direct_cost(L8, CAL) == max(4 * (8 * 16 + 48 + 3 * 8 * 9) * 100000, 2 * 3 * 8 * 16 * 9 * 500000) // 10 ** 6 + 3000000


def test_winograd_cost_by_hand():
    # 2 images, 8 -> 16 channels, 8 x 8, k = 3, pad 1, m = 2, TF32 x1: alpha 4, 16 tiles per image
    L = T.Layer(2, 8, 16, 8, 8, 3, 1, 1)
    chunk, n_chunks, cost = T.winograd_cost(L, 2, T.OPERAND_TF32, 1, CAL)
    assert (chunk, n_chunks) == (2, 1)
    v = 2 * 16 * 16 * 8 * 4
    mm = 2 * 16 * 16 * 16 * 4
    u = 16 * 16 * 8 * 4
    x = 4 * 2 * 8 * 64
    y = 4 * 2 * 16 * 64
    t_in = max(x * 100000 + v * 50000, 4 * 4 * 16 * 2 * 16 * 8 * 20000) // 10 ** 6 + 3000000
    t_con = max((v + mm) * 50000 + u * 100000, 2 * 16 * 16 * 8 * 2 * 16 * 2000) // 10 ** 6 + 3000000
    t_out = max(mm * 50000 + y * 100000, 2 * 2 * 4 * 6 * 2 * 16 * 16 * 20000) // 10 ** 6 + 3000000
    assert cost == t_in + t_con + t_out


def test_winograd_rounds_and_large_tiles_by_hand():
    """The contraction's tensor time counts full rounds of work items over the SMs, and the input transform's
    ALU term grows with alpha in the measured steps (quarters 4, 8, 9, 16).  Constants chosen so that the
    tensor and ALU terms decide: memory free, 1e9 as per tensor flop, 1e9 as per ALU flop, 7 SMs."""
    cal = [0, 0, 10 ** 9, 10 ** 9, 10 ** 9, 1000, 1 << 40, 7, 1, 1, 0, 0, 0, 0, 0, 0]
    # 1 image, 8 -> 16 channels, 4 x 4 outputs, m = 2: alpha 4, 4 tiles: 1 tile block x 1 channel block x 16
    # positions = 16 items on 7 SMs = 3 rounds
    L = T.Layer(1, 8, 16, 4, 4, 3, 1, 1)
    _, _, cost = T.winograd_cost(L, 2, T.OPERAND_TF32, 1, cal)
    flops_con = 2 * 16 * 16 * 8 * 4
    t_con = (flops_con * 10 ** 9 // 16 * 21) // 10 ** 6 + 1000
    t_in = (4 * 4 * 16 * 4 * 8 * 10 ** 9) // 10 ** 6 + 1000
    t_out = (2 * 2 * 4 * 6 * 4 * 16 * 10 ** 9) // 10 ** 6 + 1000
    assert cost == t_in + t_con + t_out
    # the same layer with 7 x 7 kernels: m = 2 -> alpha 8 (8 quarters), m = 4 -> alpha 10 (9), m = 6 -> alpha 12 (16)
    L7 = T.Layer(1, 8, 16, 12, 12, 7, 1, 3)
    for m, quarters in ((2, 8), (4, 9), (6, 16)):
        alpha = m + 6
        tiles = (12 // m) ** 2
        _, _, cost = T.winograd_cost(L7, m, T.OPERAND_TF32, 1, cal)
        items = alpha * alpha                              # 1 tile block, 1 channel block
        rounds_sms = -(-items // 7) * 7
        t_in = (quarters * alpha * alpha * alpha * tiles * 8 * 10 ** 9) // 10 ** 6 + 1000
        t_con = (2 * alpha * alpha * 16 * 8 * tiles * 10 ** 9 // items * rounds_sms) // 10 ** 6 + 1000
        t_out = (2 * m * alpha * (alpha + m) * tiles * 16 * 10 ** 9) // 10 ** 6 + 1000
        assert cost == t_in + t_con + t_out, m


def test_fused_cost_by_hand():
    L = T.Layer(2, 64, 256, 8, 8, 3, 1, 1)                 # 32 tiles: 1 tile block, 2 channel blocks, 2 K blocks
    x, y, u = 4 * 2 * 64 * 64, 4 * 2 * 256 * 64, 16 * 256 * 64 * 4
    block = max(16 * 128 * 32 * 4 * 10000 // 10 ** 6, 1000000)
    serial = 1 * (2 * block + 2000000)
    assert T.fused_cost(L, CAL) == max((x + y + u) * 100000 + x * 50000, serial * 10 ** 6) // 10 ** 6 + 3000000


def test_contraction_tiling_by_hand():
    assert T.contraction_tiling(10, 36, 512, 148) == (256, 2)
    assert T.contraction_tiling(1, 1, 64, 148) in ((64, 1), (32, 2), (16, 4))
    bn, blocks = T.contraction_tiling(98, 36, 24, 148)
    assert bn % 16 == 0 and bn * blocks >= 24


def test_first_minimum_wins_ties_and_inadmissible_is_never_chosen():
    L = T.Layer(32, 128, 128, 28, 28, 3, 1, 1)
    ppm = {key: 1 for key in ppm_table()}                   # everything admissible
    ch = T.plan(L, T.Options(), CAL, ppm)
    assert ch.cost_ps[ch.chosen] == min(ch.cost_ps)
    assert ch.chosen == ch.cost_ps.index(min(ch.cost_ps))
    ppm_bad = {key: 10 ** 9 for key in ppm}                 # nothing with rounding is admissible: only direct remains
    ch = T.plan(L, T.Options(), CAL, ppm_bad)
    assert ch.algo == T.ALGO_DIRECT and all(c == T.INADMISSIBLE for c in ch.cost_ps[1:])


def test_routing_rules():
    t = ppm_table()
    for l in all_layers():
        ch = T.plan(twin_layer(l), T.Options(), CAL, t)
        if l.k == 1:
            assert ch.algo != T.ALGO_WINOGRAD                # k = 1 "is just a matrix multiplication"
        if l.stride > 1 or l.dilation > 1 or l.groups > 1:
            assert ch.algo != T.ALGO_WINOGRAD
        if l.groups > 1:
            assert ch.algo == T.ALGO_DIRECT
    # cost never decreases with the batch
    for n in (1, 2, 4, 8, 16, 32, 64):
        a = T.plan(T.Layer(n, 64, 64, 56, 56, 3, 1, 1), T.Options(), CAL, t)
        b = T.plan(T.Layer(2 * n, 64, 64, 56, 56, 3, 1, 1), T.Options(), CAL, t)
        assert all(x <= y for x, y in zip(a.cost_ps, b.cost_ps))


def test_paper_count_on_a_worked_example():
    # Eq. 2 with o_c on its third term, times the tiles: 1 -> 1 channel, 4 x 4 input, k = 3, no padding: 2 x 2 outputs
    L = T.Layer(1, 1, 1, 4, 4, 3, 1, 0)
    assert T.paper_multiplications(L, 2) == 1 * (2 * 64 + 16 + 2 * 4 * 6)          # one 4 x 4 tile
    assert T.paper_multiplications(L, 1) == 4 * (2 * 27 + 9 + 1 * 3 * 4)           # four 3 x 3 "tiles"
    assert T.paper_choice(L)[0] == 2
    # many channels: the Hadamard term i_c o_c alpha^2 per tile dominates and the largest tile wins
    assert T.paper_choice(T.Layer(1, 512, 512, 48, 48, 3, 1, 1))[0] == 6     # 64 tiles x 64 < 144 x 36 < 576 x 16
