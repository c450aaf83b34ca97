"""Compile the CUDA sources into ``libprima.so`` next to this file (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libprima.so")
LIB_BOUNDS = os.path.join(HERE, "libprima_bounds.so")      # the same sources with -DPRIMA_BOUNDS (range-checked indices)
SOURCES = ["api.cu", "q4k_pack.cu", "q4k_gemv.cu", "q4k_gemm_tokens.cu", "finish.cu", "attention.cu", "gemv_noalloc.cu", "formats.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "-Xptxas", "-v"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "prima.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, bounds: bool = False) -> str:
    """bounds=True: the range-checked variant (an index outside its array raises bit 2 of the status word and the
    access is skipped), for tests; it is selected at run time with PRIMA_LIB=bounds."""
    LIB = LIB_BOUNDS if bounds else globals()["LIB"]
    if not force and not needs_build(LIB):
        return LIB
    objs = []
    procs = []
    bdir = "_build_bounds" if bounds else "_build"
    os.makedirs(os.path.join(HERE, bdir), exist_ok=True)
    for src in SOURCES:
        obj = os.path.join(HERE, bdir, src.replace(".cu", ".o"))
        cmd = [_nvcc()] + NVCC_FLAGS + (["-DPRIMA_BOUNDS"] if bounds else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    log = []
    for src, p in procs:
        out, _ = p.communicate()
        log.append(f"==== {src}\n{out}")
        if p.returncode != 0:
            raise RuntimeError("nvcc failed on %s:\n%s" % (src, out))
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs + ["-lcudart"], check=True)
    os.replace(tmp, LIB)
    with open(os.path.join(HERE, bdir, "ptxas.log"), "w") as f:
        f.write("\n".join(log))
    if verbose:
        print("\n".join(log))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, bounds="--bounds" in sys.argv))
