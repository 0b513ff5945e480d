"""Build libdecentlam.so (CUDA kernels + C ABI) for sm_100a, in-tree.

Usage: python -m paper_2104_11981_b200.build [--force] [--verbose]
nvcc cross-compiles without a GPU; the runtime is linked statically so the library loads
(and its host-only entry points work) on machines without a CUDA device.  Every source is
compiled to an object of its own (in parallel, only when it or a header changed), then linked.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ = os.path.join(HERE, "_build")
OUT = os.path.join(HERE, "libdecentlam.so")
SOURCES = ["api.cpp", "topology.cpp", "sharded.cpp", "step_kernels.cu", "step_merged.cu", "step_sharded.cu",
           "pmsgd_kernel.cu", "lsq_kernels.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))] + \
           [os.path.join(INCLUDE, "decentlam.h")]


def _stale() -> bool:
    if not os.path.exists(OUT):
        return True
    t = os.path.getmtime(OUT)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + _headers()
    return any(os.path.getmtime(p) > t for p in deps)


def _compile(src: str, force: bool, verbose: bool) -> str:
    obj = os.path.join(OBJ, os.path.splitext(src)[0] + ".o")
    path = os.path.join(CSRC, src)
    if not force and os.path.exists(obj):
        t = os.path.getmtime(obj)
        if all(os.path.getmtime(p) <= t for p in [path] + _headers()):
            return obj
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + ARCH + ["-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
                           "-I", INCLUDE, "-I", CSRC, "-x", "cu", "-c", path, "-o", obj]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    subprocess.run(cmd, check=True)
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return OUT
    os.makedirs(OBJ, exist_ok=True)
    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(lambda s: _compile(s, force, verbose), SOURCES))
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = OUT + ".tmp"
    subprocess.run([nvcc] + ARCH + ["-shared", "-Xcompiler", "-fPIC", "-cudart", "static"] + objs + ["-o", tmp], check=True)
    os.replace(tmp, OUT)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
