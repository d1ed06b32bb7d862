"""Build libchimera.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libchimera.so")
LIB_DEBUG = os.path.join(PKG, "libchimera_debug.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
         "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _newer(target: str, deps) -> bool:
    if not os.path.exists(target):
        return False
    t = os.path.getmtime(target)
    return all(os.path.getmtime(d) <= t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """debug=True builds libchimera_debug.so: the same sources with -DCHIMERA_DEBUG (index checks before every gather,
    guard regions in the workspace; relocatable device code because the checks share one device variable)."""
    obj_dir = OBJ + ("_debug" if debug else "")
    lib = LIB_DEBUG if debug else LIB
    flags = FLAGS + (["-DCHIMERA_DEBUG", "-rdc=true"] if debug else [])
    os.makedirs(obj_dir, exist_ok=True)
    sources = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    headers = sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + [os.path.join(ROOT, "include", "chimera.h")]
    objs, jobs = [], []
    for src in sources:
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or not _newer(obj, [src] + headers):
            cmd = [NVCC] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode:
            sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    if jobs:
        with ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            list(ex.map(run, jobs))
    if force or jobs or not _newer(lib, objs):
        tmp = lib + ".%d.tmp" % os.getpid()
        subprocess.check_call([NVCC, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
                              + (["-rdc=true"] if debug else []))
        os.replace(tmp, lib)
    return lib


def build_microbench(force: bool = False) -> str:
    """The stand-alone tensor-core instruction-rate microbenchmark (microbench/mma_rate.cu) -> build/mma_rate."""
    src = os.path.join(ROOT, "paper_2608_23553_b200", "microbench", "mma_rate.cu")
    exe = os.path.join(OBJ, "mma_rate")
    os.makedirs(OBJ, exist_ok=True)
    if force or not _newer(exe, [src, os.path.join(CSRC, "umma.cuh")]):
        subprocess.check_call([NVCC] + FLAGS + ["-o", exe, src])
    return exe


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--microbench" in sys.argv:
        print(build_microbench(force="--force" in sys.argv))
    if "--debug" in sys.argv:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug=True))
