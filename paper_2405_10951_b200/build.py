"""Builds the native library (libbsr.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbsr.so")
LIB_CHECKED = os.path.join(HERE, "libbsr_checked.so")      # the same sources with -DBSR_DEBUG: device-side index checks
SOURCES = ["engine.cu", "kernels_basic.cu", "kernels_select.cu", "gemm_simt.cu", "gemm_tc.cu", "gemm_tc2.cu", "attention_simt.cu", "attention_tc.cu", "moe.cu", "noalloc.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC",
         "--expt-relaxed-constexpr"]


def _newer(a: str, b: str) -> bool:
    return not os.path.exists(b) or os.path.getmtime(a) > os.path.getmtime(b)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Builds libbsr.so, or with checked=True libbsr_checked.so: the same sources compiled with -DBSR_DEBUG, in which
    data-dependent indices (kept / dropped token positions, expert rows) are checked on the device and a failed check
    raises a status bit that bsr_sync_status reports (nothing traps).  Select it with the environment variable
    BSR_LIBRARY=checked before the binding loads."""
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found: the native library cannot be built")
    objdir = os.path.join(HERE, "_build_checked" if checked else "_build")
    lib = LIB_CHECKED if checked else LIB
    flags = FLAGS + (["-DBSR_DEBUG"] if checked else [])
    os.makedirs(objdir, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "bsr.h"))
    objs, procs = [], []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(objdir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _newer(s, o) or any(_newer(hf, o) for hf in headers):
            cmd = [nvcc, *flags, "-c", s, "-o", o] + (["-Xptxas", "-v"] if verbose else [])
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src} ---\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if procs or not os.path.exists(lib):
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib, *objs, "-lcudart"])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
