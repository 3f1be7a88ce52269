"""Builds the C-ABI shared library with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2002_12418_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
BUILD = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libmnnconv_b200.so")
SOURCES = ["api.cu", "calibrate.cu", "contract_umma.cu", "contract_pair.cu", "wino_fused.cu", "strassen.cu", "implicit_gemm.cu", "wino_rect.cu", "gather_direct.cu", "wino_transforms.cu", "wino_inst_k2.cu", "wino_inst_a4_6.cu",
           "wino_inst_a8.cu", "wino_inst_a10.cu", "wino_inst_a12.cu",
           "generator.cpp", "planner.cpp"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _local_includes(path: str, seen: set) -> None:
    """Collects, recursively, the files `path` includes with quotes (headers of this repo only)."""
    if path in seen or not os.path.exists(path):
        return
    seen.add(path)
    with open(path, errors="replace") as f:
        for line in f:
            s = line.strip()
            if s.startswith("#include \""):
                name = s.split('"')[1]
                _local_includes(os.path.normpath(os.path.join(os.path.dirname(path), name)), seen)


def _newest_dependency(src: str) -> float:
    """mtime of the newest of the source and every repo header it reaches (after a change of the compiler
    flags in this file, build with --force)."""
    seen: set = set()
    _local_includes(os.path.join(CSRC, src), seen)
    return max(os.path.getmtime(p) for p in seen)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(BUILD, exist_ok=True)
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []
    rebuilt = []

    def compile_one(src: str) -> str:
        obj = os.path.join(BUILD, os.path.splitext(src)[0] + ".o")
        if not force and os.path.exists(obj) and os.path.getmtime(obj) >= _newest_dependency(src):
            return obj
        rebuilt.append(src)
        cmd = [nvcc] + NVCC_FLAGS + extra + ["-x", "cu", "-c", os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed on " + src)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    if not rebuilt and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(o) for o in objs):
        return LIB
    tmp = LIB + ".tmp%d" % os.getpid()
    cmd = [nvcc, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("link failed")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
