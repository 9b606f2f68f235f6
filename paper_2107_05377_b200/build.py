"""Builds the C-ABI library (csrc/*.cu -> libmt_bert.so next to this file) for sm_100a.

nvcc cross-compiles without a GPU.  Run as ``python -m paper_2107_05377_b200.build``.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmt_bert.so")
SOURCES = ["mt_api.cu", "gemm_tcgen05.cu", "attention.cu", "attention_tc.cu", "gemm_ln_tcgen05.cu", "gemm_ln_wide_tcgen05.cu", "rowwise.cu", "noalloc.cu", "wait_probe.cu"]


def sources():
    return [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + [os.path.join(CSRC, "mt_kernels.h"), os.path.join(CSRC, "tc_ptx.cuh"), os.path.join(CSRC, "rowwise.cuh"), os.path.join(CSRC, "cluster_ptx.cuh"), os.path.join(HERE, "..", "include", "mt_bert.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    tmp = f"{LIB}.{os.getpid()}.tmp"   # built aside and renamed, so a concurrent loader never sees a partial file
    cmd = [nvcc, "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "--threads", "4", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-o", tmp] + sources()
    if verbose:
        cmd += ["-Xptxas", "-v"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed building libmt_bert.so")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
