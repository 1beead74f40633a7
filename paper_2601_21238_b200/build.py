"""Build libstwq.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a, and, when its source
directory is present, the optional companion libstwq_mc.so (the GEMM variant that shares an
operand between CTA pairs by cluster multicast; single-GPU builds only)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libstwq.so")
CSRC_MC = os.path.join(HERE, "csrc_mc")
LIB_MC = os.path.join(HERE, "libstwq_mc.so")
BUILD_DIR = os.path.join(HERE, "_build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--ftz=false", "--prec-div=true",
    "--prec-sqrt=true", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.sep not in c or os.path.exists(c)):
            return c
    return "nvcc"


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def sources_mc():
    return sorted(glob.glob(os.path.join(CSRC_MC, "*.cu")))


def _stale(lib, srcs) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = srcs + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def needs_build() -> bool:
    return _stale(LIB, sources()) or (bool(sources_mc()) and _stale(LIB_MC, sources_mc()))


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ and link them into libstwq.so next to this file; likewise
    csrc_mc/ into libstwq_mc.so if that directory is there."""
    if force or _stale(LIB, sources()):
        _build_one(sources(), LIB, verbose)
    if sources_mc() and (force or _stale(LIB_MC, sources_mc())):
        _build_one(sources_mc(), LIB_MC, verbose)
    return LIB


def _build_one(srcs, lib, verbose):
    os.makedirs(BUILD_DIR, exist_ok=True)
    objs = []
    procs = []
    for src in srcs:
        obj = os.path.join(BUILD_DIR, os.path.basename(src)[:-3] + ".o")
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode != 0:
            sys.stderr.write(out)
        failed |= pr.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = lib + ".tmp%d" % os.getpid()
    subprocess.run([_nvcc(), "-arch=sm_100a", "-shared", "-o", tmp] + objs + ["-Xcompiler", "-fPIC"], check=True)
    os.replace(tmp, lib)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
