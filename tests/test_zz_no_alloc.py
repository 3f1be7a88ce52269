"""The run that allocates nothing (mnn_conv_run_static) against mnn_conv_run.

Some users of the library are given their tensors by a host application and may not
create device memory themselves (a plug-in under another framework's memory budget, a
real-time loop that must not make calls which can block on the driver).  For them the
library carries a fixed built-in workspace.  This file checks, through the C ABI, that a
layer run on that built-in workspace gives bit for bit the result of the same plan run on
a caller-provided workspace (the kernels are deterministic, so anything but equality would
be a fault) and meets the accuracy class against the fp64 oracle — several calls in a row
with different layers, because the built-in array is shared and keeps the previous call's
contents, among them a layer whose channel padding must be zero-filled on the dirty array
— and that a plan too large for it is refused.  It is collected last so that a failure here cannot hide other tests.
"""
import numpy as np
import pytest

from oracle import direct_conv as oc
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import assert_close, to_dev

pytestmark = pytest.mark.gpu


def _both_ways(torch, layer, opts):
    x, w, b = W.make_inputs(layer)
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad,
                          layer.dilation, opts)
    assert 0 < r.info.workspace_bytes <= B.STATIC_WORKSPACE_BYTES
    xd, wd, bd = to_dev(torch, x), to_dev(torch, w), to_dev(torch, b)
    y_ref = r.run(xd, wd, bd)                                    # existing entry point, caller's workspace
    torch.cuda.synchronize()
    assert r.device_status() == 0
    y_new = torch.full_like(y_ref, float("nan"))
    B.mnn_conv_run_static(r.plan, xd.data_ptr(), wd.data_ptr(), bd.data_ptr() if bd is not None else None,
                          y_new.data_ptr(), r.stream())
    torch.cuda.synchronize()
    ref, got = y_ref.cpu().numpy(), y_new.cpu().numpy()
    r.close()
    assert np.array_equal(got, ref), "the static run differs from the run on a caller's workspace"
    want = oc.direct_conv(x, w, b, layer.stride, layer.pad, layer.dilation, layer.groups, layer.relu)
    assert_close(got, want, B.PREC_TF32, layer.name + " against the oracle")
    return got, ref


def test_static_workspace_run_matches_workspace_run_twice():
    import torch
    assert torch.cuda.is_available()
    B.lib()
    # first call: tensor-core contraction, BF16 hi + lo operands
    a = W.ConvLayer("a", 2, 48, 40, 20, 20, 3, 1, 1, relu=True, seed=901)
    got, ref = _both_ways(torch, a, B.make_opts(relu=1, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=B.OPERAND_BF16,
                                                passes=3))
    assert_close(got, ref, B.PREC_TF32, "first call")
    # second call right after it: another shape and format on the same (now dirty) array
    b = W.ConvLayer("b", 3, 24, 72, 13, 13, 3, 1, 1, relu=True, seed=902)
    got, ref = _both_ways(torch, b, B.make_opts(relu=1, force_algo=B.ALGO_WINOGRAD, force_m=2, operand=B.OPERAND_TF32,
                                                passes=1))
    assert_close(got, ref, B.PREC_TF32, "second call")
    # and the GEMM scheme, whose contraction writes y directly
    c = W.ConvLayer("c", 2, 32, 48, 15, 15, 3, 2, 1, relu=True, seed=903)
    got, ref = _both_ways(torch, c, B.make_opts(relu=1, force_algo=B.ALGO_GEMM, operand=B.OPERAND_TF32))
    assert_close(got, ref, B.PREC_TF32, "third call")
    # a channel count that is not a multiple of 8: the padding columns of U and V must be written as zeros
    # over whatever the larger layers above left in the array
    d = W.ConvLayer("d", 2, 20, 40, 11, 11, 3, 1, 1, relu=True, seed=904)
    _both_ways(torch, d, B.make_opts(relu=1, force_algo=B.ALGO_WINOGRAD, force_m=4, operand=B.OPERAND_BF16, passes=3))
    # the single-kernel Winograd path keeps only its packed weights in the array
    e = W.ConvLayer("e", 2, 24, 136, 12, 12, 3, 1, 1, relu=True, seed=905)
    _both_ways(torch, e, B.make_opts(relu=1, fused=B.FUSED_ONLY))


def test_static_workspace_rejects_plans_that_do_not_fit():
    import torch
    big = W.ConvLayer("big", 32, 256, 256, 56, 56, 3, 1, 1, seed=1)
    plan = B.mnn_conv_plan_ex(big.N, big.Cin, big.Cout, big.H, big.W, 3, 1, 1, 1,
                              B.make_opts(relu=1, force_algo=B.ALGO_WINOGRAD, force_m=4))
    assert B.mnn_conv_plan_query(plan).workspace_bytes > B.STATIC_WORKSPACE_BYTES
    t = torch.zeros(64, device="cuda:0")
    with pytest.raises(B.MnnError) as ei:
        B.mnn_conv_run_static(plan, t.data_ptr(), t.data_ptr(), None, t.data_ptr() + 64, 0)
    assert ei.value.code == B.MNN_EWORKSPACE and "built-in workspace" in str(ei.value)
    B.mnn_conv_destroy(plan)
