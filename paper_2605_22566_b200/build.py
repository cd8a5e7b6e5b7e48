"""Builds the CUDA libraries in-tree with nvcc for sm_100a (no JIT cache, no torch extension).

  libgfpath.so  the path-attention library (C ABI of include/gf.h)
  libgfgen.so   device copy of the synthetic input generator (test/bench inputs only)
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libgfpath.so")
GEN_PATH = os.path.join(HERE, "libgfgen.so")

ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]
PATH_SOURCES = ["api.cu", "tables.cu", "kvpool.cu", "decode.cu", "extend_tc.cu", "pruning.cu", "residual_encode.cu", "debug.cu", "scoring.cu"]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    raise RuntimeError("nvcc not found")


def _newer(target: str, deps) -> bool:
    if not os.path.exists(target):
        return False
    t = os.path.getmtime(target)
    return all(os.path.getmtime(d) <= t for d in deps)


def _run(cmd):
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("build failed: " + " ".join(cmd) + "\n" + r.stdout + r.stderr)
    return r.stdout + r.stderr


def build(force: bool = False, verbose: bool = False, ptxas_info: bool = False) -> None:
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(INCLUDE, "gf.h"))
    extra = ["-Xptxas", "-v"] if ptxas_info else []
    user_flags = os.environ.get("GF_NVCC_FLAGS", "").split()  # e.g. -DGF_DEBUG_BOUNDS; forces a rebuild
    extra += user_flags
    force = force or bool(user_flags)

    def compile_one(src):
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src.replace(".cu", ".o"))
        if force or ptxas_info or not _newer(o, [s] + headers):
            out = _run([nvcc] + ARCH + FLAGS + extra + ["-c", s, "-o", o])
            if verbose or ptxas_info:
                print(out, file=sys.stderr)
        return o

    with ThreadPoolExecutor(max_workers=6) as ex:
        objs = list(ex.map(compile_one, PATH_SOURCES + ["gen.cu"]))
    path_objs, gen_obj = objs[:-1], objs[-1]
    if force or not _newer(LIB_PATH, path_objs):
        _run([nvcc] + ARCH + ["-shared", "-o", LIB_PATH] + path_objs + ["-lcudart"])
    if force or not _newer(GEN_PATH, [gen_obj]):
        _run([nvcc] + ARCH + ["-shared", "-o", GEN_PATH, gen_obj, "-lcudart"])


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas" in sys.argv)
    print("built", LIB_PATH, GEN_PATH)
