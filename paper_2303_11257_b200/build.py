"""Builds libunitscale.so in-tree with nvcc for sm_100a.

    python -m paper_2303_11257_b200.build [--force]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libunitscale.so")
SOURCES = ["host.cu", "elementwise.cu", "softmax.cu", "layernorm.cu", "diagnostics.cu", "gemm.cu", "gemm_group.cu", "ffn_hidden.cu", "static_ws.cu", "attention.cu"]
# (operand bytes, A MN-major, B MN-major): forward, backward-input, backward-weight for FP8 and 16-bit operands
GEMM_PARTS = [(1, 0, 1), (1, 0, 0), (1, 1, 1), (2, 0, 1), (2, 0, 0), (2, 1, 1)]
HEADERS = ["common.cuh", "rowwise.cuh", "sm100.cuh", "gemm_kernel.cuh", "gemm_group.cuh", "gemm_launch.h", "gemm_inst.cu", "host.h", os.path.join("..", "..", "include", "unitscale.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(args):
    res = subprocess.run(args, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(args) + "\n" + res.stdout + res.stderr)
    return res.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path.

    Every translation unit is compiled to an object in parallel (gemm_inst.cu once per operand
    width and layout), then linked into libunitscale.so next to this file."""
    if not force and not _stale():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    common = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v" if verbose else "-O3", "-c"]
    jobs, objs = [], []
    for f in SOURCES:
        o = os.path.join(objdir, f.replace(".cu", ".o"))
        objs.append(o)
        jobs.append(common + ["-o", o, os.path.join(CSRC, f)])
    for es, amn, bmn in GEMM_PARTS:
        o = os.path.join(objdir, f"gemm_inst_{es}_{amn}_{bmn}.o")
        objs.append(o)
        jobs.append(common + [f"-DUS_INST_ES={es}", f"-DUS_INST_AMN={amn}", f"-DUS_INST_BMN={bmn}", "-o", o,
                              os.path.join(CSRC, "gemm_inst.cu")])
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as pool:
        logs = list(pool.map(_compile, jobs))
    _compile([_nvcc(), "-shared", "-o", LIB] + objs + ["-lcudart"])
    if verbose:
        print("\n".join(logs))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
