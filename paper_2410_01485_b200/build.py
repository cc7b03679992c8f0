"""Builds the CUDA library in-tree with nvcc for sm_100a (no GPU needed to compile)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "liblg_sparse_attn.so")
LIB_DEBUG = os.path.join(HERE, "liblg_sparse_attn_debug.so")   # -DLG_DEBUG: schedule reads bounds-checked
SOURCES = ["lg_api.cu", "lg_fwd.cu", "lg_bwd.cu", "lg_decode.cu", "lg_host_step.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "-Xptxas", "-v", "-DLG_NVTX"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _newer(a: str, b: str) -> bool:
    return (not os.path.exists(b)) or os.path.getmtime(a) > os.path.getmtime(b)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile the library in-tree.  debug=True builds the checked variant (LG_DEBUG) beside it."""
    sub = "_build_debug" if debug else "_build"
    lib = LIB_DEBUG if debug else LIB
    flags = NVCC_FLAGS + (["-DLG_DEBUG"] if debug else [])
    os.makedirs(os.path.join(HERE, sub), exist_ok=True)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "lg.h")]
    objs, jobs = [], []
    for src in SOURCES:
        obj = os.path.join(HERE, sub, src.replace(".cu", ".o"))
        objs.append(obj)
        if force or any(_newer(d, obj) for d in deps):
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        cmd = [_nvcc(), *flags, "-c", os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, res.stdout, res.stderr))
        with open(obj + ".ptxas.log", "w") as f:
            f.write(res.stderr)
        if verbose:
            sys.stderr.write(res.stderr)

    with ThreadPoolExecutor(max_workers=4) as pool:
        list(pool.map(compile_one, jobs))
    if jobs or force or not os.path.exists(lib):
        cmd = [_nvcc(), "-shared", "-o", lib, *objs, "-Xcompiler", "-fPIC", "-cudart", "static"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("link failed:\n%s\n%s" % (res.stdout, res.stderr))
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
