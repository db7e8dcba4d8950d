"""Builds the C-ABI library `libmetis_b200.so` in-tree with nvcc for sm_100a.

Usage: python -m paper_2509_00404_b200.build [--force]
"""
import concurrent.futures
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libmetis_b200.so")
SOURCES = ["api.cu", "quantize.cu", "gemm_check.cu", "gemm_tcgen05.cu", "split.cu", "coeff_tc.cu", "residual_tc.cu", "linear.cu", "static_ws.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
         "--fmad=true", "-Xptxas", "-v"]


def _nvcc():
    return shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"


def _sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _stale():
    if not os.path.exists(LIB) or not os.path.exists(LIB_DEBUG):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(PKG, "..", "include", "metis.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


LIB_DEBUG = os.path.join(PKG, "libmetis_b200_debug.so")      # the same sources with METIS_DEBUG_BUILD (index checks on every output store)


def _compile(job):
    src, debug = job
    obj = os.path.join(OBJ + ("_debug" if debug else ""), src.replace(".cu", ".o"))
    cmd = [_nvcc(), *FLAGS, *(["-DMETIS_DEBUG_BUILD"] if debug else []), "-c", os.path.join(CSRC, src), "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    with open(obj + ".log", "w") as f:
        f.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s" % (src, r.stderr[-4000:]))
    return obj


def build(force=False):
    if not force and not _stale():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    os.makedirs(OBJ + "_debug", exist_ok=True)
    jobs = [(s_, dbg) for dbg in (False, True) for s_ in _sources()]
    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        objs = list(ex.map(_compile, jobs))
    n = len(_sources())
    for lib, group in ((LIB, objs[:n]), (LIB_DEBUG, objs[n:])):
        cmd = [_nvcc(), "-shared", "-o", lib, *group, "-gencode", "arch=compute_100a,code=sm_100a"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n" + r.stderr[-4000:])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
