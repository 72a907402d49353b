"""Compile the C checker with gcc into oracle/liba2cid2_oracle.so (test infrastructure)."""
from __future__ import annotations

import os
import subprocess
import threading

_LOCK = threading.Lock()  # the checker's column-parallel runs may ask for the library from several threads at once

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "a2cid2_oracle.c")
LIB = os.path.join(HERE, "liba2cid2_oracle.so")


def build(force: bool = False) -> str:
    with _LOCK:
        return _build(force)


def _build(force: bool) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    # -ffp-contract=off: every product and sum is rounded on its own, as written.
    cmd = ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
