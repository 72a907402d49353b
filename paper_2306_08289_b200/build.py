"""Compile the CUDA library for sm_100a into paper_2306_08289_b200/liba2cid2.so (in-tree).

Extra nvcc flags for experiments may be given in the environment variable A2CID2_NVCC_FLAGS, e.g.
"-DA2_EVENT_THREADS=512" (threads per CTA of the event kernel) or "-DA2_TUNING_KNOBS=1" (a build whose
launch shapes can be overridden from the environment, see csrc/a2cid2_internal.h). The default build has
no such flags and reads no tuning variable at run time."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(HERE, "liba2cid2.so")
SOURCES = ["api.cu", "kernels.cu", "scheduler.cpp", "spectral.cpp"]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return cand


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "a2cid2.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC,-O2,-Wall", "-shared", "-cudart", "static",
           "-I", INCLUDE, "-I", CSRC, "-o", tmp]
    cmd += os.environ.get("A2CID2_NVCC_FLAGS", "").split()  # extra flags for experiments, e.g. -DA2_EVENT_THREADS=512
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("nvcc failed")
    if verbose:
        sys.stderr.write(r.stdout + r.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
