"""Build the CUDA library in-tree: csrc/*.cu, csrc/*.cpp -> libgett_b200.so (sm_100a).

Sources named *_mc.cu (the CTA-pair variant of the tensor-core kernel) go into a library of
their own, libgett_b200_mc.so, which the main library loads if it is there; a tree without
those sources builds and runs the same, without the variant."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libgett_b200.so")
LIB_MC = os.path.join(HERE, "libgett_b200_mc.so")
LIB_BENCH = os.path.join(HERE, "libgett_b200_bench.so")  # measurement helpers (*_bench.cu), not the product
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMMON = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC,-fvisibility=hidden",
          "-I", os.path.join(os.path.dirname(HERE), "include")]


def sources():
    return sorted(f for f in os.listdir(CSRC)
                  if f.endswith((".cu", ".cpp")) and not f.endswith(("_mc.cu", "_bench.cu")))


def sources_mc():
    return sorted(f for f in os.listdir(CSRC) if f.endswith("_mc.cu"))


def _newest_header() -> float:
    t = 0.0
    for d in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(d):
            if f.endswith((".h", ".cuh")) or (d == CSRC and f == "kernel_umma.cu"):  # (included by *_mc.cu)
                t = max(t, os.path.getmtime(os.path.join(d, f)))
    return t


def _compile(src: str, verbose: bool) -> str:
    obj = os.path.join(OBJ, src + ".o")
    path = os.path.join(CSRC, src)
    if os.path.exists(obj) and os.path.getmtime(obj) >= max(os.path.getmtime(path), _newest_header()):
        return obj
    cmd = [NVCC, *ARCH, *COMMON, "-c", path, "-o", obj]
    if src.endswith(".cu") and verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    if src.endswith(".cpp"):
        cmd = [NVCC, *COMMON, "-x", "c++", "-c", path, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
    if verbose and (r.stdout or r.stderr):
        sys.stderr.write(f"--- {src}\n{r.stdout}{r.stderr}")
    return obj


def build(verbose: bool = False, force: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    if force:
        for f in os.listdir(OBJ):
            os.remove(os.path.join(OBJ, f))
    srcs = sources()
    with ThreadPoolExecutor(max_workers=min(8, len(srcs))) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose), srcs))
    _link(LIB, objs)
    mc = sources_mc()
    if mc:
        _link(LIB_MC, [_compile(s, verbose) for s in mc])
    elif os.path.exists(LIB_MC):
        os.remove(LIB_MC)
    bench = sorted(f for f in os.listdir(CSRC) if f.endswith("_bench.cu"))
    if bench:
        _link(LIB_BENCH, [_compile(s, verbose) for s in bench])
    return LIB


def _link(lib: str, objs) -> None:
    if not os.path.exists(lib) or any(os.path.getmtime(o) > os.path.getmtime(lib) for o in objs):
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.check_call([NVCC, *ARCH, "-shared", "-o", tmp, *objs, "-lcudart_static",
                               "-Xlinker", "--exclude-libs=ALL"])
        os.replace(tmp, lib)


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv, force="-f" in sys.argv))
