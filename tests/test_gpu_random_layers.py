"""Seeded random layers through the C ABI against the CPU oracle: shapes nobody picked by hand.  Every layer runs
with the planner's own choice and with the schemes that can be forced on its kind; a forced scheme the library
declines for the shape (MnnError) is skipped.  Tolerances as in test_gpu_parity.py; the sliding-window kernels
accumulate in fp32 and are held to 1e-6."""
import random

import numpy as np
import pytest

from oracle import direct_conv as oc
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import max_abs_frac, rel_l2, to_dev

pytestmark = pytest.mark.gpu

KINDS = ["winograd", "pointwise", "gemm", "depthwise", "few_channels", "grouped"]


def draw_layer(rng, kind, case):
    N = rng.choice([1, 2, 3, 5, 8])
    stride, dil, groups = 1, 1, 1
    if kind == "winograd":
        k = rng.choice([3, 3, 3, 5, 7, 2])
        H, Wd = rng.randint(k, 40), rng.randint(k, 40)
        Cin = rng.choice([3, 8, 16, 20, 32, 48, 64, 72, 96, 128, 136])
        Cout = rng.choice([8, 16, 24, 32, 64, 80, 128, 144, 272])
        pad = rng.choice([0, (k - 1) // 2, (k - 1) // 2])
    elif kind == "pointwise":
        k, pad = 1, 0
        H, Wd = rng.randint(2, 40), rng.randint(2, 40)
        Cin = rng.choice([8, 24, 32, 40, 64, 100, 128, 256, 512])
        Cout = rng.choice([8, 16, 40, 64, 128, 136, 256, 300, 512])
    elif kind == "gemm":
        k, stride, dil = rng.choice([1, 3, 3, 5, 7]), rng.choice([1, 2, 2, 3]), rng.choice([1, 1, 2])
        pad = rng.randint(0, k // 2 + 1)
        H, Wd = rng.randint(dil * (k - 1) + 1, 36), rng.randint(dil * (k - 1) + 1, 36)
        Cin, Cout = rng.choice([3, 8, 16, 32, 64, 96]), rng.choice([8, 16, 32, 64, 100])
    elif kind == "depthwise":
        k, pad, stride = 3, 1, rng.choice([1, 2])
        Cin = Cout = groups = rng.choice([1, 3, 8, 13, 32, 64, 100])
        H, Wd = rng.randint(1, 60), rng.randint(1, 70)
    elif kind == "few_channels":
        k, stride = rng.choice([3, 3, 3, 5, 7]), rng.choice([1, 2, 2])
        pad = rng.choice([0, 1, k // 2])
        Cin, Cout = rng.choice([1, 2, 3, 3, 3, 4]), rng.choice([8, 16, 32, 33, 64, 70])
        H = 2 * rng.randint((k + 1) // 2, 32) if rng.random() < 0.5 else rng.randint(k, 64)
        Wd = rng.choice([rng.randint(k, 64), 4 * rng.randint(2, 16)])
    else:
        k, stride, dil, pad = rng.choice([1, 2, 3, 5]), rng.choice([1, 2]), rng.choice([1, 2]), rng.randint(0, 2)
        groups = rng.choice([2, 4])
        Cin, Cout = groups * rng.choice([1, 2, 4, 8, 16]), groups * rng.choice([1, 2, 4, 8, 16])
        H, Wd = rng.randint(dil * (k - 1) + 1, 30), rng.randint(dil * (k - 1) + 1, 30)
    if (H + 2 * pad - dil * (k - 1) - 1) // stride + 1 < 1 or (Wd + 2 * pad - dil * (k - 1) - 1) // stride + 1 < 1:
        return None
    return W.ConvLayer("r%d" % case, N, Cin, Cout, H, Wd, k, stride, pad, dil, groups=groups, relu=rng.random() < 0.5,
                       seed=case)


def forced_variants(rng, kind, layer):
    v = [dict()]
    if kind == "winograd" and layer.k in (3, 5):
        v.append(dict(force_algo=B.ALGO_WINOGRAD, force_m=rng.choice([2, 4, 6])))
    if kind == "winograd" and layer.k == 3 and layer.pad <= 2:
        v.append(dict(fused=B.FUSED_ONLY))
    if kind in ("pointwise", "gemm"):
        v.append(dict(force_algo=B.ALGO_GEMM))
    if kind == "gemm" and layer.k > 1:
        v.append(dict(force_algo=B.ALGO_GEMM, gemm_lhs=B.GEMM_LHS_IMPLICIT))
    if kind in ("depthwise", "few_channels", "grouped"):
        v.append(dict(force_algo=B.ALGO_DIRECT))
    return v


@pytest.mark.parametrize("kind", KINDS)
def test_random_layers(kind):
    import torch
    assert torch.cuda.is_available()
    B.lib()
    rng = random.Random(KINDS.index(kind) + 101)
    ran = 0
    for case in range(14):
        layer = draw_layer(rng, kind, 1000 * KINDS.index(kind) + case)
        if layer is None:
            continue
        x, w, b = W.make_inputs(layer)
        ref = oc.direct_conv(x, w, b, layer.stride, layer.pad, layer.dilation, layer.groups, layer.relu)
        for forced in forced_variants(rng, kind, layer):
            opts = B.make_opts(groups=layer.groups, relu=layer.relu, **forced)
            try:
                r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad,
                                      layer.dilation, opts)
            except B.MnnError:
                assert forced, "the planner's own choice must exist for %r" % (layer,)
                continue
            y = r.run(to_dev(torch, x), to_dev(torch, w), to_dev(torch, b))
            torch.cuda.synchronize()
            status, info, got = r.device_status(), r.info, y.cpu().numpy()
            r.close()
            what = "%r forced %r -> algo %d m %d lhs %d fused %d" % (layer, forced, info.algo, info.m, info.gemm_lhs, info.fused)
            assert status == 0, what
            assert got.shape == ref.shape and np.isfinite(got).all(), what
            assert rel_l2(got, ref) <= (1e-6 if info.algo == B.ALGO_DIRECT else 1e-3), what
            assert max_abs_frac(got, ref) <= 2e-2, what
            ran += 1
    assert ran >= 14
