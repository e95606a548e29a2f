"""Compile the CUDA library (sm_100a) into paper_2511_15898_b200/libgr_b200.so."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgr_b200.so")
LIB_CHECK = os.path.join(HERE, "libgr_b200_check.so")      # the bounds-checked build (-DGR_CHECK)
OBJ = os.path.join(HERE, "_build")
SOURCES = ["gr_api.cu", "gr_alpha.cu", "gr_static.cu", "gr_scan.cu", "gr_solve.cu", "gr_fast.cu", "gr_fast_n4.cu", "gr_fast_n8.cu",
           "gr_fast_n16.cu", "gr_fast_w8.cu", "gr_fast_w16.cu", "gr_fullsort.cu", "gr_verify.cu"]
HEADERS = [os.path.join(CSRC, "gr_common.cuh"), os.path.join(CSRC, "gr_prep.cuh"), os.path.join(CSRC, "gr_fast.cuh"), os.path.join(CSRC, "gr_verify.cuh"), os.path.join(CSRC, "gr_host.h"),
           os.path.join(ROOT, "include", "gr.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build(check: bool = False) -> bool:
    lib = LIB_CHECK if check else LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Compile each source to an object (in parallel; objects newer than every source and header are kept),
    then link the shared library.  check=True builds the bounds-checked variant (-DGR_CHECK: every access through a
    pointer into shared memory, the workspace records or the params block is range-checked, an out-of-range access
    is skipped and reported as status GR_CHECK_FAILED) into a library file of its own; it is for tests only."""
    LIB = LIB_CHECK if check else globals()["LIB"]
    OBJ = globals()["OBJ"] + ("_check" if check else "")
    if not force and not needs_build(check):
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    flags = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if check:
        flags += ["-DGR_CHECK"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    hdr_time = max(os.path.getmtime(h) for h in HEADERS)
    jobs = []
    objs = []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(OBJ, s[:-3] + ".o")
        objs.append(obj)
        fresh = (not force and not verbose and os.path.exists(obj)
                 and os.path.getmtime(obj) > max(os.path.getmtime(src), hdr_time))
        if not fresh:
            jobs.append((s, subprocess.Popen([_nvcc()] + flags + ["-c", src, "-o", obj], stdout=subprocess.PIPE,
                                             stderr=subprocess.STDOUT, text=True)))
    failed = []
    for s, proc in jobs:
        out, _ = proc.communicate()
        if verbose:
            sys.stderr.write(out)
        if proc.returncode != 0:
            failed.append(s + ":\n" + out)
    if failed:
        raise RuntimeError("nvcc failed:\n" + "\n".join(failed))
    res = subprocess.run([_nvcc(), "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a"]
                         + objs + ["-ldl", "-o", LIB], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
