"""Planner validation: for every layer of a workload, time each scheme the planner considers
admissible and print it next to the planner's predicted cost and choice.

    python -m paper_2002_12418_b200.sweep --workload config4_b64 [--calibrate] [--reps 5]

One JSON line per layer: the candidate table (predicted microseconds from the integer cost
model, measured microseconds of mnn_conv_run with prepared weights, L2 flushed before every
run), the planner's choice, the fastest measured candidate and their ratio.  With
--calibrate the cost constants are first measured on this GPU (mnn_calibrate) and printed.
"""
from __future__ import annotations

import argparse
import json
import statistics

from . import binding as B
from . import workloads as W

CANDIDATES = ([("direct", B.ALGO_DIRECT, 0, 0, 0), ("gemm tf32", B.ALGO_GEMM, 0, B.OPERAND_TF32, 1),
               ("gemm bf16", B.ALGO_GEMM, 0, B.OPERAND_BF16, 1)]
              + [("wino m%d tf32x1" % m, B.ALGO_WINOGRAD, m, B.OPERAND_TF32, 1) for m in (2, 4, 6)]
              + [("wino m%d tf32x3" % m, B.ALGO_WINOGRAD, m, B.OPERAND_TF32, 3) for m in (2, 4, 6)]
              + [("wino m%d bf16x1" % m, B.ALGO_WINOGRAD, m, B.OPERAND_BF16, 1) for m in (2, 4, 6)]
              + [("wino m%d bf16x3" % m, B.ALGO_WINOGRAD, m, B.OPERAND_BF16, 3) for m in (2, 4, 6)])


def workload(name: str):
    table = {"config0": W.config0, "config1_b1": lambda: W.config1(1), "config1_b32": lambda: W.config1(32),
             "config2_b1": lambda: W.config2(1), "config2_b32": lambda: W.config2(32),
             "config3_b1": lambda: W.config3(1), "config3_b64": lambda: W.config3(64),
             "config4_b64": lambda: W.config4(64)}
    return table[name]()


def time_plan(torch, layer, opts, xd, wd, bd, reps, flush):
    r = B.ConvLayerRunner(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad,
                          layer.dilation, opts)
    y = torch.empty((layer.N, layer.Cout, r.info.OH, r.info.OW), device=xd.device)
    r.prepare(wd)
    r.run(xd, wd, bd, y)
    ms = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        r.run(xd, wd, bd, y)
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    status = r.device_status()
    info = r.info
    r.close()
    return statistics.median(ms) * 1e3, status, info


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="config4_b64")
    ap.add_argument("--precision", default="tf32", choices=["tf32", "bf16"])
    ap.add_argument("--calibrate", action="store_true")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--layers", default="", help="comma-separated layer indices (default: all)")
    args = ap.parse_args()
    import torch
    B.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    if args.calibrate:
        consts = B.mnn_calibrate(0, torch.cuda.current_stream().cuda_stream)
        print(json.dumps({"calibration": consts}))
    else:
        print(json.dumps({"calibration": B.mnn_get_calibration(), "note": "built-in defaults or last record set"}))
    cls = B.PREC_TF32 if args.precision == "tf32" else B.PREC_BF16
    layers = workload(args.workload)
    if args.layers:
        layers = [layers[int(i)] for i in args.layers.split(",")]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for layer in layers:
        x, w, b = W.make_inputs(layer)
        xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
        bd = torch.from_numpy(b).to(dev) if b is not None else None
        plan = B.mnn_conv_plan_ex(layer.N, layer.Cin, layer.Cout, layer.H, layer.W, layer.k, layer.stride, layer.pad,
                                  layer.dilation, B.make_opts(groups=layer.groups, relu=layer.relu, precision=cls))
        info = B.mnn_conv_plan_query(plan)
        B.mnn_conv_destroy(plan)
        rows = []
        for i, (name, algo, m, operand, passes) in enumerate(CANDIDATES):
            cost = info.cost_ps[i]
            if cost == B.COST_INADMISSIBLE:
                continue
            o = B.make_opts(groups=layer.groups, relu=layer.relu, precision=cls, force_algo=algo, force_m=m,
                            operand=operand, passes=passes)
            us, status, _ = time_plan(torch, layer, o, xd, wd, bd, args.reps, flush)
            rows.append({"candidate": name, "predicted_us": round(cost / 1e6, 2), "measured_us": round(us, 2),
                         "device_status": status, "chosen": i == info.chosen_candidate})
        best = min(rows, key=lambda r: r["measured_us"])
        chosen = next(r for r in rows if r["chosen"])
        print(json.dumps({"layer": layer.name, "N": layer.N, "candidates": rows, "chosen": chosen["candidate"],
                          "fastest": best["candidate"],
                          "chosen_over_fastest": round(chosen["measured_us"] / best["measured_us"], 3),
                          "direct_equiv_TFLOPs_chosen": round(layer.direct_flops / chosen["measured_us"] / 1e6, 1)}))
        del xd, wd, bd
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
