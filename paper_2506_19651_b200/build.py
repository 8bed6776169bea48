"""Build the CUDA library in-tree: paper_2506_19651_b200/libpevlm.so (sm_100a only).

    python -m paper_2506_19651_b200.build [--force]

nvcc cross-compiles without a GPU.  The library links the CUDA runtime statically, so it
has no dependency on a particular libcudart at load time.
"""
from __future__ import annotations

import os
import subprocess
import sys

_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_DIR, "csrc")
LIB = os.path.join(_DIR, "libpevlm.so")
SOURCES = ["api.cu", "rope_kernel.cu", "assemble_kernel.cu", "attn_kernel.cu", "merge_kernel.cu", "query_noalloc.cu", "selftest.cu"]
HEADERS = ["internal.h", "ptx.cuh", os.path.join("..", "..", "include", "pevlm.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC", "-cudart", "static"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    # PEVLM_TRACE=1: time stamps of the kernel's hand-offs, read by timeline.py (include/pevlm_trace.h)
    extra = ["-DPEVLM_TRACE"] if os.environ.get("PEVLM_TRACE") == "1" else []
    if not force and not _stale():
        return LIB
    objs = []
    build_dir = os.path.join(_DIR, "build")
    os.makedirs(build_dir, exist_ok=True)
    procs = []
    for src in SOURCES:
        obj = os.path.join(build_dir, src.replace(".cu", ".o"))
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        procs.append((cmd, subprocess.Popen(cmd)))
        objs.append(obj)
    for cmd, pr in procs:
        if pr.wait() != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    tmp = LIB + f".tmp{os.getpid()}"
    link = [_nvcc(), "-shared", *NVCC_FLAGS[:2], "-cudart", "static", "-o", tmp, *objs]
    subprocess.run(link, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
