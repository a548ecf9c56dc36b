"""Builds ``libpatdnn.so`` in-tree with nvcc for sm_100a (no torch involved)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpatdnn.so")
SOURCES = ["api.cu", "kernels_simple.cu", "kernels_tiled.cu", "umma_conv.cu", "umma_chain.cu", "prun_conv.cu", "prun_plan.cpp", "smallc_split.cu", "smallc_jit.cu", "tiled_inst_4x8.cu",
           "tiled_inst_4x4.cu", "tiled_inst_2x8.cu", "fkw_encoder.cpp", "tiled_plan.cpp"]
HEADERS = ["kernels.hpp", "umma_ptx.cuh", "kernels_tiled.cuh", "fkw_encoder.hpp", os.path.join("generated", "tiled_cases.inc"),
           os.path.join("..", "..", "include", "patdnn.h")]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--threads", "0"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu/.cpp under csrc/ into one shared library; returns its path."""
    sys.path.insert(0, CSRC)
    import gen_cases                     # writes csrc/generated/tiled_cases.inc (the PTX FMA bodies)
    gen_cases.generate()
    if not force and not needs_build():
        return LIB
    objs = []
    objdir = os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    procs = []
    for s in SOURCES:
        o = os.path.join(objdir, s + ".o")
        objs.append(o)
        src = os.path.join(CSRC, s)
        if not force and os.path.exists(o) and os.path.getmtime(o) > max(
                os.path.getmtime(src), *(os.path.getmtime(os.path.join(CSRC, h)) for h in HEADERS)):
            continue
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-x", "cu", "-c", src, "-o", o]
        procs.append((s, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for s, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(out)
        if p.returncode:
            raise RuntimeError(f"nvcc failed on {s}")
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-ldl"])   # cudart static; driver API via entry points
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
