"""Runs ONE convolution layer a few times through the C ABI: a small, self-ending
command to put under a profiler or to time stage by stage.

    python -m paper_2002_12418_b200.profile_case --N 16 --C 256 --H 56 --k 3 --m 4 \
        --operand bf16 --passes 3 [--stages input] [--reps 3] [--algo winograd]

Prints one JSON line with the plan's decisions and, per stage, the mean kernel
time over the repetitions (CUDA events around every launch), the algorithmic
bytes and flops and the rates they imply.  Inputs are seeded N(0,1) draws.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as B

STAGES = {"weight": B.STAGE_WEIGHT, "input": B.STAGE_INPUT, "contract": B.STAGE_CONTRACT, "output": B.STAGE_OUTPUT,
          "all": B.STAGE_INPUT | B.STAGE_CONTRACT | B.STAGE_OUTPUT}
OPERANDS = {"auto": B.OPERAND_AUTO, "tf32": B.OPERAND_TF32, "bf16": B.OPERAND_BF16, "fp32ref": B.OPERAND_FP32_REF}
LHS = {"auto": B.GEMM_LHS_AUTO, "patches": B.GEMM_LHS_PATCHES, "x": B.GEMM_LHS_X, "implicit": B.GEMM_LHS_IMPLICIT}
ALGOS = {"auto": B.ALGO_AUTO, "winograd": B.ALGO_WINOGRAD, "gemm": B.ALGO_GEMM, "direct": B.ALGO_DIRECT}


def stage_work(info, N, Cin, Cout, H, W, k, groups):
    """Algorithmic bytes and tensor flops of each stage of one run (what the kernels must move)."""
    x_bytes = 4 * N * Cin * H * W
    y_bytes = 4 * N * Cout * info.OH * info.OW
    b_el = (2 if info.operand == B.OPERAND_BF16 else 4) * (2 if info.passes == 3 else 1)
    out = {}
    if info.algo == B.ALGO_WINOGRAD and info.fused:
        T = N * (-(-info.OH // 2)) * (-(-info.OW // 2))
        out["contract"] = (x_bytes + y_bytes + 4 * 16 * Cout * Cin, 2 * 16 * Cout * Cin * T)
    elif info.algo == B.ALGO_WINOGRAD:
        a2 = info.alpha ** 2
        T = N * (-(-info.OH // info.m)) * (-(-info.OW // info.m))
        v, mm, u = b_el * a2 * Cin * T, 4 * a2 * Cout * T, b_el * a2 * Cout * Cin
        out["input"] = (x_bytes + v, 0)
        out["contract"] = (v + mm + u * info.n_chunks, 2 * a2 * Cout * Cin * T * info.passes)
        out["output"] = (mm + y_bytes, 0)
    elif info.algo == B.ALGO_GEMM and info.strassen:
        T, Kh, Mh = N * info.OH * info.OW // 2, Cin // 2, Cout // 2
        v, mm = b_el * 7 * T * Kh, 4 * 7 * Mh * T
        out["input"] = (x_bytes + v, 0)
        out["contract"] = (v + mm + b_el * 7 * Mh * Kh, 2 * 7 * Mh * Kh * T * info.passes)
        out["output"] = (mm + y_bytes, 0)
    elif info.algo == B.ALGO_GEMM:
        K, T = Cin * k * k, N * info.OH * info.OW
        v = b_el * T * K
        if info.gemm_lhs in (B.GEMM_LHS_X, B.GEMM_LHS_IMPLICIT):
            v = x_bytes                    # the contraction reads x itself
        else:
            out["input"] = (x_bytes + v, 0)
        out["contract"] = (v + b_el * Cout * K + y_bytes, 2 * T * Cout * K * info.passes)
    else:
        out["contract"] = (x_bytes + y_bytes + 4 * Cout * (Cin // groups) * k * k,
                           2 * N * Cout * (Cin // groups) * info.OH * info.OW * k * k)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--N", type=int, default=16)
    ap.add_argument("--C", type=int, default=256, help="Cin (and Cout unless --Cout)")
    ap.add_argument("--Cout", type=int, default=0)
    ap.add_argument("--H", type=int, default=56)
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--pad", type=int, default=-1, help="default (k-1)/2")
    ap.add_argument("--groups", type=int, default=1)
    ap.add_argument("--m", type=int, default=0)
    ap.add_argument("--operand", default="auto", choices=sorted(OPERANDS))
    ap.add_argument("--passes", type=int, default=0)
    ap.add_argument("--algo", default="auto", choices=sorted(ALGOS))
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--lhs", default="auto", choices=sorted(LHS), help="left operand of the GEMM scheme")
    ap.add_argument("--precision", default="tf32", choices=["tf32", "bf16"])
    ap.add_argument("--stages", default="all", choices=sorted(STAGES))
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--flush", action="store_true", help="write 256 MB between repetitions")
    ap.add_argument("--strassen", type=int, default=0, help="1: one Strassen level on a 1x1 layer's product")
    ap.add_argument("--fused", type=int, default=0, help="0 planner, 1 never, 2 the single-kernel F(2x2,3x3) path")
    args = ap.parse_args()

    import torch
    B.lib()
    dev = torch.device("cuda:0")
    Cin, Cout = args.C, args.Cout or args.C
    pad = (args.k - 1) // 2 if args.pad < 0 else args.pad
    o = B.make_opts(groups=args.groups, relu=1, precision=B.PREC_TF32 if args.precision == "tf32" else B.PREC_BF16,
                    operand=OPERANDS[args.operand], passes=args.passes, force_algo=ALGOS[args.algo], force_m=args.m,
                    chunk_images=args.chunk, gemm_lhs=LHS[args.lhs], fused=args.fused, strassen=args.strassen)
    r = B.ConvLayerRunner(args.N, Cin, Cout, args.H, args.H, args.k, args.stride, pad, 1, o)
    info = r.info
    g = torch.Generator(device="cpu").manual_seed(1)
    x = torch.randn((args.N, Cin, args.H, args.H), generator=g).to(dev)
    w = (torch.randn((Cout, Cin // args.groups, args.k, args.k), generator=g) / np.sqrt(Cin * args.k * args.k)).to(dev)
    b = torch.randn((Cout,), generator=g).to(dev)
    y = torch.empty((args.N, Cout, info.OH, info.OW), device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if args.flush else None
    r.run(x, w, b, y)                      # weights prepared, every buffer written once
    torch.cuda.synchronize()
    B.mnn_conv_profile(r.plan, True)
    names = ["weight", "input", "contract", "output"]
    tot = [0.0] * 4
    cnt = [0] * 4
    mask = STAGES[args.stages] if info.algo != B.ALGO_DIRECT else B.STAGE_CONTRACT
    for _ in range(args.reps):
        if flush is not None:
            flush.zero_()
        r.run(x, w, b, y, stage_mask=mask)
        ms, n = B.mnn_conv_profile_read(r.plan)
        for i in range(4):
            tot[i] += ms[i]
            cnt[i] += n[i]
    torch.cuda.synchronize()
    status = r.device_status()
    work = stage_work(info, args.N, Cin, Cout, args.H, args.H, args.k, args.groups)
    stages = {}
    for i, nm in enumerate(names):
        if cnt[i] == 0 or nm not in work:
            continue
        ms = tot[i] / args.reps
        by, fl = work[nm]
        stages[nm] = {"ms": round(ms, 5), "launches_per_run": cnt[i] // args.reps, "bytes": by,
                      "GBps": round(by / ms / 1e6, 1), "tensor_TFLOPs": round(fl / ms / 1e9, 1) if fl else None}
    total_ms = sum(s["ms"] for s in stages.values())
    direct = 2 * args.N * Cout * (Cin // args.groups) * info.OH * info.OW * args.k * args.k
    print(json.dumps({"algo": B.ALGO_NAMES[info.algo], "m": info.m, "operand": B.OPERAND_NAMES[info.operand],
                      "passes": info.passes, "gemm_lhs": info.gemm_lhs, "fused": info.fused, "strassen": info.strassen, "chunk_images": info.chunk_images, "n_chunks": info.n_chunks,
                      "workspace_MB": round(info.workspace_bytes / 2 ** 20, 1), "device_status": status,
                      "stages": stages, "sum_ms": round(total_ms, 5),
                      "direct_equiv_TFLOPs": round(direct / total_ms / 1e9, 1) if total_ms > 0 else None}))
    r.close()


if __name__ == "__main__":
    main()
