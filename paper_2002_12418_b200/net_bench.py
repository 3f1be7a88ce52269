"""Preparation-execution decoupling at network level (Section 3.2 of the paper, its Table 2) on this GPU:
the MobileNet-v1 conv stack (27 layers) run (a) layer by layer from Python, each layer with its own plan and
workspace, (b) as ONE mnn_net_run over a shared workspace, (c) as a CUDA-graph replay of that call.

    python -m paper_2002_12418_b200.net_bench [--batch 1] [--reps 50]

Prints one JSON line with the three times per forward pass (CUDA events, median), the launches per pass and
the workspace sizes with and without sharing."""
from __future__ import annotations

import argparse
import json
import statistics

from . import binding as B
from . import workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--reps", type=int, default=50)
    ap.add_argument("--calibration", default="measure", choices=["measure", "builtin"],
                    help="builtin plans from the library's frozen record (use it under a profiler, which slows "
                         "the calibration's own launches)")
    args = ap.parse_args()
    import torch
    B.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    N = args.batch
    layers = W.config3(N)
    if args.calibration == "measure":
        B.mnn_calibrate(0, torch.cuda.current_stream().cuda_stream)
    x = torch.from_numpy(W.make_inputs(layers[0])[0]).to(dev)
    ws, bs = [], []
    for l in layers:
        _, w, b = W.make_inputs(l.with_batch(1))
        ws.append(torch.from_numpy(w).to(dev))
        bs.append(torch.from_numpy(b).to(dev))

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        out = []
        for _ in range(args.reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1))
        return statistics.median(out)

    # (a) layer by layer
    runners, acts = [], [x]
    for l, w in zip(layers, ws):
        r = B.ConvLayerRunner(N, l.Cin, l.Cout, l.H, l.W, l.k, l.stride, l.pad, l.dilation,
                              B.make_opts(groups=l.groups, relu=l.relu))
        r.prepare(w)
        runners.append(r)
        acts.append(torch.empty((N, l.Cout, r.info.OH, r.info.OW), device=dev))

    def per_layer():
        for i, r in enumerate(runners):
            r.run(acts[i], ws[i], bs[i], acts[i + 1])

    ms_layers = timed(per_layer)
    y_layers = acts[-1].clone()

    # (b) one call
    net = B.NetRunner(N, 224, 224, layers)
    net.prepare(ws)
    net.bind(ws, bs)
    y = torch.empty_like(y_layers)
    ms_net = timed(lambda: net.run(x, y))
    same = bool(torch.equal(y, y_layers))

    # (c) CUDA graph of that call
    side = torch.cuda.Stream(dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        net.run(x, y)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            net.run(x, y)
    torch.cuda.synchronize()
    ms_graph = timed(graph.replay)
    same_graph = bool(torch.equal(y, y_layers))
    status = net.device_status()
    flops = sum(l.direct_flops for l in layers)
    print(json.dumps({"workload": "MobileNet-v1 conv stack", "batch": N, "layers": len(layers),
                      "launches_per_pass": net.info.launches_per_run,
                      "ms_layer_by_layer": round(ms_layers, 4), "ms_net_run": round(ms_net, 4),
                      "ms_graph_replay": round(ms_graph, 4),
                      "direct_equiv_TFLOPs_graph": round(flops / ms_graph / 1e9, 2),
                      "same_result_net": same, "same_result_graph": same_graph, "device_status": status,
                      "workspace_MB_shared": round(net.info.workspace_bytes / 2 ** 20, 1),
                      "workspace_MB_per_layer_sum": round(net.info.sum_of_layer_workspaces / 2 ** 20, 1),
                      "activation_buffer_MB": round(net.info.activation_bytes / 2 ** 20, 1)}))


if __name__ == "__main__":
    main()
