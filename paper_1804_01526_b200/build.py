"""Builds the CUDA library in-tree: ``python -m paper_1804_01526_b200.build``.

nvcc cross-compiles for sm_100a without a GPU. The shared object is written next to this
file (``libhbfp.so``) so that it travels with the source tree.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhbfp.so")
SOURCES = ["api.cu", "quantize.cu", "gemm_simt.cu", "gemm_small.cu", "gemm_tc.cu", "gemm_tc2.cu", "gemm_conv.cu", "gemm_static.cu"]
# (object name, source, extra flags): quantize.cu is compiled a second time for the full-tile kernel of small tiles
EXTRA_OBJECTS = [("quantize_tiles_small.o", "quantize.cu", ["-DHBFP_QUANT_PART=2", "-Xptxas", "-O1"])]
# Per-file additions. The paired-SM GEMM is built with ptxas -O1: measured in SM cycles per launch (16384^3, b = 128)
# 8.57 M against 8.86 M at the default level, and 12 % / 9 % fewer cycles for blocks of 64 / 32; the other files were
# measured too and are a toss-up kernel by kernel (single-SM GEMM: 8-bit + 9 %, 12-bit - 6 %), so they keep the default.
EXTRA_FLAGS = {"gemm_tc2.cu": ["-Xptxas", "-O1"],
               "gemm_conv.cu": ["-Xptxas", "-O1"]}      # 128-channel forward 16.0 -> 15.0 us, 64-channel unchanged

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC,-fvisibility=hidden",
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true",   # never fast-math: parity is bit-exact
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "hbfp.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or _stale()):
        return LIB
    objdir = os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    procs = []
    objs = []
    for src in SOURCES:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        objs.append(obj)
        cmd = ["nvcc", *NVCC_FLAGS, *EXTRA_FLAGS.get(src, []), "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for obj_name, src, flags in EXTRA_OBJECTS:
        obj = os.path.join(objdir, obj_name)
        objs.append(obj)
        cmd = ["nvcc", *NVCC_FLAGS, *flags, "-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((obj_name, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.run(["nvcc", "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
                    "-cudart", "static"], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
