"""Builds the sm_100a shared library (librk.so) in-tree with nvcc.  No JIT cache: the built
file sits next to the sources so that it travels with the repository snapshot."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "librk.so")
CHECK_LIB_PATH = os.path.join(LIB_DIR, "librk_check.so")   # the same sources with -DRK_CHECK (device index checks)
SOURCES = ["rk_host.cu", "rk_attn.cu", "rk_gemm.cu", "rk_stream.cu", "rk_policy.cu"]
HEADERS = ["rk_ptx.cuh", "rk_internal.h", os.path.join("..", "..", "include", "rk.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, s) for s in _sources()] + [os.path.join(CSRC, h) for h in HEADERS]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def build_library(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """check=True builds librk_check.so: the same sources with -DRK_CHECK, whose kernels test every index they
    derive from a request table and report a bad one through the status word (a debugging aid for small cases)."""
    out_path = CHECK_LIB_PATH if check else LIB_PATH
    if not force and not needs_build() and os.path.exists(out_path) and \
            os.path.getmtime(out_path) >= os.path.getmtime(LIB_PATH):
        return out_path
    os.makedirs(LIB_DIR, exist_ok=True)
    objs = []
    procs = []
    for src in _sources():
        obj = os.path.join(LIB_DIR, src.replace(".cu", "_check.o" if check else ".o"))
        cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
               "-Xcompiler", "-fPIC", "-c", os.path.join(CSRC, src), "-o", obj]
        if check:
            cmd.append("-DRK_CHECK")
        if verbose:
            cmd += ["-Xptxas", "-v"]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(f"--- {src} ---\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    link = [_nvcc(), "-shared", "-o", out_path] + objs
    r = subprocess.run(link, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout)
        raise RuntimeError("link failed")
    return out_path


def ensure_built() -> str:
    """Builds the library if the built file is not there (a fresh checkout); an existing build is left alone.
    A missing compiler is an error: nothing else can compute the path."""
    return LIB_PATH if os.path.exists(LIB_PATH) else build_library(force=True)


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, check="--check" in sys.argv))
