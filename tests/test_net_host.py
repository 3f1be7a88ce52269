"""Host side of the network-level plan (no GPU): the virtual walk's memory layout."""
import pytest

from paper_2002_12418_b200 import binding as B
from paper_2002_12418_b200 import workloads as W


def test_mobilenet_stack_layout_shares_the_transient_part():
    layers = W.config3(64)
    net = B.mnn_net_plan(64, 224, 224, layers)
    info = B.mnn_net_query(net)
    assert info.n_layers == len(layers) == 27
    assert (info.out_C, info.out_H, info.out_W) == (1024, 7, 7)
    # every layer's output extent matches the workload's own arithmetic
    for i, l in enumerate(layers):
        assert (info.OH[i], info.OW[i]) == (l.OH, l.OW)
        assert info.algo[i] in (B.ALGO_WINOGRAD, B.ALGO_GEMM, B.ALGO_DIRECT)
    # layout: persistent parts + one shared transient part + two activation buffers
    assert info.workspace_bytes == info.persistent_bytes + info.transient_bytes + 2 * info.activation_bytes
    largest_act = max(4 * 64 * l.Cout * l.OH * l.OW for l in layers[:-1])
    assert largest_act <= info.activation_bytes < largest_act + 1024
    # sharing never costs: persistent + one transient part is at most the per-layer workspaces added up (equal when
    # no layer of the stack needs a transient part, e.g. when every GEMM reads x itself or gathers implicitly)
    assert info.persistent_bytes + info.transient_bytes <= info.sum_of_layer_workspaces
    B.mnn_net_destroy(net)


def test_channel_mismatch_and_limits_are_rejected():
    a = W.ConvLayer("a", 1, 8, 16, 12, 12, 3, 1, 1)
    b = W.ConvLayer("b", 1, 24, 16, 12, 12, 3, 1, 1)          # Cin != previous Cout
    with pytest.raises(B.MnnError) as e:
        B.mnn_net_plan(1, 12, 12, [a, b])
    assert "layer 1" in str(e.value)
    with pytest.raises(B.MnnError):
        B.mnn_net_plan(1, 12, 12, [])
    net = B.mnn_net_plan(1, 12, 12, [a])
    with pytest.raises(B.MnnError) as e:
        B.mnn_net_set_workspace(net, 0, 0)
    assert e.value.code == B.MNN_EWORKSPACE
    B.mnn_net_destroy(net)
