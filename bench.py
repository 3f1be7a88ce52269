#!/usr/bin/env python
"""Benchmark of the convolution hot path on B200.

A step = one forward pass of every layer of the workload (ResNet-18-style 3x3
stride-1 layers at batch 32: weights already transformed, inputs resident in HBM)
through mnn_conv_run.  Prints ONE JSON line: direct-convolution-equivalent TFLOP/s,
ms per step, the roofline position of the dominant kernel, the end-to-end figure with
host buffers, and the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload config1_b32]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "conv TFLOP/s (direct-conv-equivalent)"
UNIT = "TFLOP/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch (mean over the four layers of one step) from one ncu
# capture of this file's default workload (profiles/bench_config1_b32_launch_list.md gives the command).  Valid
# for config1_b32 / tf32 and the kernels as captured; set an entry to None when its kernel changes.
NCU_DRAM_BYTES_PER_LAUNCH = {"config1_b32/tf32": {"input": 40.30e6, "contraction": 45.51e6, "output": 15.49e6}}


def workload_layers(name: str):
    from paper_2002_12418_b200 import workloads as W
    table = {
        "config1_b32": lambda: W.config1(32),
        "config1_b1": lambda: W.config1(1),
        "config2_b32": lambda: W.config2(32),
        "config3_b64": lambda: W.config3(64),
        "config4_b64": lambda: W.config4(64),
    }
    if name not in table:
        raise SystemExit("unknown workload %s (have %s)" % (name, ", ".join(sorted(table))))
    return table[name]()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------
# Clock sampling during the timed region.
# ---------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        clocks, maxes, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm, mx = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            if t0 - 0.05 <= ts <= t1 + 0.2:
                clocks.append(sm)
                maxes.append(mx)
                for nm, val in zip(names, parts[2:6]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
        if not clocks:
            for ts, line in self.lines[-3:]:
                parts = [p.strip() for p in line.split(",")]
                try:
                    clocks.append(float(parts[0]))
                    maxes.append(float(parts[1]))
                except (ValueError, IndexError):
                    pass
        return {"sm_mhz": statistics.median(clocks) if clocks else None,
                "sm_max_mhz": max(maxes) if maxes else None, "reasons": sorted(reasons), "samples": len(clocks)}


# ---------------------------------------------------------------------------
# CPU oracle timing (the cpu_baseline leg and --impl reference).
# ---------------------------------------------------------------------------
def time_oracle_sample(layers, images=4, min_seconds=0.0):
    """The fp64 direct-convolution oracle, as it stands, on the first `images` images of every
    layer, repeated until `min_seconds` of CPU work have been timed."""
    from oracle import direct_conv as oc
    from paper_2002_12418_b200 import workloads as W
    import numpy as np
    total_flops, total_s = 0, 0.0
    inputs = []
    for layer in layers:
        part = layer.with_batch(min(images, layer.N))
        inputs.append((part, W.make_inputs(part)))
    while True:
        for part, (x, w, b) in inputs:
            t0 = time.perf_counter()
            y = oc.direct_conv(x, w, b, part.stride, part.pad, part.dilation, part.groups, part.relu)
            total_s += time.perf_counter() - t0
            total_flops += part.direct_flops
            assert np.isfinite(y).all()
        if total_s >= min_seconds:
            break
    return total_flops, total_s, oc.threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers = workload_layers(args.workload)
    from oracle import direct_conv as oc
    oc.build()
    for _ in range(min(args.warmup, 1)):
        time_oracle_sample(layers[:1])
    flops, secs = 0, 0.0
    cores = 1
    for _ in range(args.steps):
        f, s, cores = time_oracle_sample(layers)
        flops += f
        secs += s
    value = flops / secs / 1e12
    sample = "first 4 images of each of the %d layers per step (%.3f GFLOP direct per step), fp64 nested loops" % (
        len(layers), flops / args.steps / 1e9)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": args.workload, "note": "CPU oracle on a bounded sample of the workload"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# Algorithmic bytes / flops per stage of one layer (what the kernels must move).
# ---------------------------------------------------------------------------
def stage_work(layer, info):
    from paper_2002_12418_b200 import binding as B
    N, Cin, Cout = layer.N, layer.Cin, layer.Cout
    x_bytes = 4 * N * Cin * layer.H * layer.W
    y_bytes = 4 * N * Cout * info.OH * info.OW
    b_el = (2 if info.operand == B.OPERAND_BF16 else 4) * (2 if info.passes == 3 else 1)
    out = {}
    if info.algo == B.ALGO_WINOGRAD:
        a2 = info.alpha ** 2
        th, tw = -(-info.OH // info.m), -(-info.OW // info.m)
        T = N * th * tw
        v_bytes = b_el * a2 * Cin * T
        m_bytes = 4 * a2 * Cout * T
        u_bytes = b_el * a2 * Cout * Cin
        out["input"] = {"bytes": x_bytes + v_bytes, "flops": 0}
        out["contraction"] = {"bytes": v_bytes + m_bytes + u_bytes * info.n_chunks,
                              "flops": 2 * a2 * Cout * Cin * T * info.passes}
        out["output"] = {"bytes": m_bytes + y_bytes, "flops": 0}
    elif info.algo == B.ALGO_GEMM:
        K = Cin * layer.k ** 2
        T = N * info.OH * info.OW
        v_bytes = b_el * T * K
        out["input"] = {"bytes": x_bytes + v_bytes, "flops": 0}
        out["contraction"] = {"bytes": v_bytes + b_el * Cout * K + y_bytes, "flops": 2 * T * Cout * K * info.passes}
    else:
        w_bytes = 4 * Cout * (Cin // layer.groups) * layer.k ** 2
        out["contraction"] = {"bytes": x_bytes + y_bytes + w_bytes, "flops": layer.direct_flops}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config1_b32")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--precision", default="tf32", choices=["tf32", "bf16"])
    ap.add_argument("--launch", default="graph", choices=["graph", "stream"],
                    help="how a timed step is issued: one CUDA-graph replay of the step's launches (captured "
                         "once from the same C-ABI calls), or the calls themselves on the stream")
    ap.add_argument("--calibration", default="measure", choices=["measure", "builtin"],
                    help="measure: run mnn_calibrate on this GPU before planning (default); builtin: plan from the "
                         "library's frozen B200 record (use under a profiler, which slows the calibration launches)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import numpy as np
    import torch
    from paper_2002_12418_b200 import binding as B
    from paper_2002_12418_b200 import replicas as R
    from paper_2002_12418_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    B.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    layers = workload_layers(args.workload)
    prec = B.PREC_TF32 if args.precision == "tf32" else B.PREC_BF16
    # pre-inference: the planner's cost constants are measured once on this GPU, before any plan is made
    if args.calibration == "measure":
        calibration = B.mnn_calibrate(local_rank, torch.cuda.current_stream(dev).cuda_stream)
        torch.cuda.synchronize(dev)
    else:
        calibration = B.mnn_get_calibration()
    # every rank works on its own batch of the same shape (weak scaling; images are independent)
    state = []
    for i, layer in enumerate(layers):
        lay = layer if world == 1 else layer.with_batch(layer.N, seed_offset=R.rank_seed_offset(rank))
        x, w, b = W.make_inputs(lay)
        o = B.make_opts(groups=lay.groups, relu=lay.relu, precision=prec)
        r = B.ConvLayerRunner(lay.N, lay.Cin, lay.Cout, lay.H, lay.W, lay.k, lay.stride, lay.pad, lay.dilation, o,
                              device=str(dev))
        xd = torch.from_numpy(x).to(dev)
        wd = torch.from_numpy(w).to(dev)
        bd = torch.from_numpy(b).to(dev) if b is not None else None
        yd = torch.empty((lay.N, lay.Cout, r.info.OH, r.info.OW), dtype=torch.float32, device=dev)
        r.prepare(wd)
        state.append({"layer": lay, "runner": r, "x": xd, "w": wd, "b": bd, "y": yd, "x_host": x})
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    def one_step():
        for s in state:
            s["runner"].run(s["x"], s["w"], s["b"], s["y"])

    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        one_step()
    barrier()
    for s in state:
        assert s["runner"].device_status() == 0, "a kernel reported a bounded wait that ran out"

    # The step's launches captured once into a CUDA graph: the same C-ABI calls, recorded instead of run.
    # Replaying it issues the same kernels with the same arguments without the per-launch host work.
    timed_step = one_step
    if args.launch == "graph":
        step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(step_graph):
            one_step()
        timed_step = step_graph.replay
        for _ in range(3):
            flush.zero_()
            timed_step()
        barrier()

    # ---- timed region: K steps, L2 flushed before each, device time by CUDA events ----
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier()
    t_wall0 = time.time()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for k in range(args.steps):
        flush.zero_()
        ev[k][0].record(stream)
        timed_step()
        ev[k][1].record(stream)
    barrier()
    t_wall1 = time.time()
    step_ms = [a.elapsed_time(b) for a, b in ev]
    clocks = sampler.stop(t_wall0, t_wall1)
    total_ms = float(sum(step_ms))
    total_ms = R.max_over_ranks(dist, total_ms, dev)
    flops_step = sum(s["layer"].direct_flops for s in state)
    value = R.whole_job_throughput(flops_step, args.steps, world, total_ms)
    launches = sum(s["runner"].info.launches_per_run for s in state) * args.steps

    # ---- per-kernel durations (events around every launch), same steps again ----
    stage_names = ["weight", "input", "contraction", "output"]
    stage_ms = {n: 0.0 for n in stage_names}
    stage_n = {n: 0 for n in stage_names}
    stage_bytes = {n: 0 for n in stage_names}
    stage_flops = {n: 0 for n in stage_names}
    per_layer = []
    for s in state:
        B.mnn_conv_profile(s["runner"].plan, True)
    for k in range(args.steps):
        flush.zero_()
        one_step()
        for s in state:
            ms, n = B.mnn_conv_profile_read(s["runner"].plan)
            work = stage_work(s["layer"], s["runner"].info)
            for i, nm in enumerate(stage_names):
                stage_ms[nm] += ms[i]
                stage_n[nm] += n[i]
                if n[i] and nm in work:
                    stage_bytes[nm] += work[nm]["bytes"]
                    stage_flops[nm] += work[nm]["flops"]
            if k == args.steps - 1:
                info = s["runner"].info
                per_layer.append({"name": s["layer"].name, "algo": B.ALGO_NAMES[info.algo], "m": info.m,
                                  "operand": B.OPERAND_NAMES[info.operand], "passes": info.passes,
                                  "chunk_images": info.chunk_images, "stage_ms_last_step": [round(v, 4) for v in ms]})
    for s in state:
        B.mnn_conv_profile(s["runner"].plan, False)
    torch.cuda.synchronize(dev)
    peaks = measured_peaks()
    dominant = max(stage_names, key=lambda n: stage_ms[n])
    dom_launches = max(stage_n[dominant], 1)
    dom_ms = stage_ms[dominant] / dom_launches
    dom_bytes = stage_bytes[dominant] / dom_launches
    achieved_gbs = dom_bytes / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
    roofline = {"kernel": dominant, "bound": "hbm", "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved_gbs / peaks["hbm_gbs"],
                "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get("%s/%s" % (args.workload, args.precision), {}).get(dominant),
                "algorithmic_bytes_per_launch": dom_bytes, "peak_source": peaks["source"],
                "avg_launch_us": dom_ms * 1e3, "launches": stage_n[dominant],
                "stage_ms_per_step": {n: stage_ms[n] / args.steps for n in stage_names},
                "stage_gbs": {n: (stage_bytes[n] / (stage_ms[n] * 1e-3) / 1e9 if stage_ms[n] > 0 else None)
                              for n in stage_names},
                "contraction_tflops": (stage_flops["contraction"] / (stage_ms["contraction"] * 1e-3) / 1e12
                                       if stage_ms["contraction"] > 0 else None)}

    # ---- end to end through the public call with HOST buffers ----
    h2d = sum(s["x_host"].nbytes for s in state)
    d2h = sum(s["y"].numel() * 4 for s in state)
    for s in state:
        s["x_pin"] = torch.from_numpy(s["x_host"]).pin_memory()
        s["y_pin"] = torch.empty(s["y"].shape, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))

    # Three streams, linked by events: the copy of layer i + 1's input and the read-back of layer i - 1's
    # result run while layer i computes (the GPU's copy engines work in both directions at once).
    h2d_stream, d2h_stream = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    for s in state:
        s["x_ready"], s["x_free"] = torch.cuda.Event(), torch.cuda.Event()
        s["y_ready"], s["y_free"] = torch.cuda.Event(), torch.cuda.Event()
        s["x_free"].record(stream)
        s["y_free"].record(stream)

    def e2e_step():
        for s in state:
            with torch.cuda.stream(h2d_stream):
                h2d_stream.wait_event(s["x_free"])               # the previous pass over this layer has read x
                s["x"].copy_(s["x_pin"], non_blocking=True)
                s["x_ready"].record(h2d_stream)
            stream.wait_event(s["x_ready"])
            stream.wait_event(s["y_free"])                       # the previous result has been read back
            s["runner"].run(s["x"], s["w"], s["b"], s["y"])
            s["x_free"].record(stream)
            s["y_ready"].record(stream)
            with torch.cuda.stream(d2h_stream):
                d2h_stream.wait_event(s["y_ready"])
                s["y_pin"].copy_(s["y"], non_blocking=True)
                s["y_free"].record(d2h_stream)

    def e2e_join():
        for s in state:
            stream.wait_event(s["y_free"])

    e2e_step()
    e2e_join()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e2e_join()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = R.max_over_ranks(dist, e2e_ms, dev)
    e2e_value = R.whole_job_throughput(flops_step, e2e_steps, world, e2e_ms)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        f, secs, cores = time_oracle_sample(layers, images=4, min_seconds=10.0)
        cpu_baseline = {"value": f / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": "first 4 images of each of the %d layers, repeated for %.1f s (%.1f GFLOP direct in "
                                  "all), fp64 nested loops" % (len(layers), secs, f / 1e9)}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "tf32" if prec == B.PREC_TF32 else "bf16",
                "data": "synthetic",
                "config": {"workload": args.workload, "layers": len(layers), "batch_per_gpu": layers[0].N,
                           "l2": "flushed before every step (256 MB write)", "weights": "pre-transformed",
                           "launch": "CUDA graph replay per step" if args.launch == "graph" else "C-ABI calls on the stream",
                           "accuracy_class": args.precision, "planner_calibration": calibration[:9], "calibration_source": args.calibration, "plans": per_layer},
                "clocks": clocks, "roofline": roofline,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "ms_per_step": e2e_ms / e2e_steps},
                "gpu_launches": launches, "cpu_baseline": cpu_baseline}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
