"""GPU parity of the network-level plan: a whole stack of layers through ONE mnn_net_run, against the fp64
oracle applied layer after layer to the same seeded inputs.

Tolerance: every layer meets relative L2 <= 1e-3 against an exact evaluation of ITS input (class TF32).
Through a stack the deviations can at most add up, so after L layers the bound is L * 1e-3 (written below);
max-abs keeps the per-layer bound 2e-2 * max|y_ref|."""
import numpy as np
import pytest

from oracle import direct_conv as oc
from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W
from tests.util import TOL_MAX_ABS_FRAC, rel_l2, max_abs_frac, to_dev

pytestmark = pytest.mark.gpu


def oracle_chain(layers, x, ws, bs):
    a = x
    for l, w, b in zip(layers, ws, bs):
        a = oc.direct_conv(a.astype(np.float32), w, b, l.stride, l.pad, l.dilation, l.groups, l.relu)
    return a


def run_net(layers, N, H):
    import torch
    B.lib()
    x = W.make_inputs(layers[0].with_batch(N))[0]
    ws, bs = [], []
    for l in layers:
        _, w, b = W.make_inputs(l.with_batch(1))
        ws.append(w)
        bs.append(b)
    r = B.NetRunner(N, H, H, layers)
    wd, bd = [to_dev(torch, w) for w in ws], [to_dev(torch, b) for b in bs]
    r.prepare(wd)
    r.bind(wd, bd)
    y1 = r.run(to_dev(torch, x))
    y2 = r.run(to_dev(torch, x))              # a second pass re-uses every buffer
    torch.cuda.synchronize()
    assert r.device_status() == (0, -1)
    assert torch.equal(y1, y2)
    info = r.info
    got = y1.cpu().numpy()
    r.close()
    return got, oracle_chain(layers, x, ws, bs), info


def test_mobilenet_v1_stack_batch2():
    layers = W.config3(2)
    got, ref, info = run_net(layers, 2, 224)
    assert got.shape == ref.shape == (2, 1024, 7, 7)
    assert np.isfinite(got).all()
    assert rel_l2(got, ref) <= len(layers) * 1e-3
    assert max_abs_frac(got, ref) <= TOL_MAX_ABS_FRAC
    algos = {info.algo[i] for i in range(info.n_layers)}
    assert B.ALGO_DIRECT in algos                      # depthwise layers


def test_stack_of_3x3_layers_goes_through_winograd():
    chans = [32, 64, 64, 128, 128]
    layers = [W.ConvLayer("s%d" % i, 8, chans[i], chans[i + 1], 28, 28, 3, 1, 1, seed=700 + i) for i in range(4)]
    got, ref, info = run_net(layers, 8, 28)
    assert rel_l2(got, ref) <= len(layers) * 1e-3
    assert max_abs_frac(got, ref) <= TOL_MAX_ABS_FRAC
    assert any(info.algo[i] == B.ALGO_WINOGRAD for i in range(info.n_layers))
    assert info.persistent_bytes + info.transient_bytes < info.sum_of_layer_workspaces
