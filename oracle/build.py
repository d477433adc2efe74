"""Compile the C oracle into oracle/libfff_oracle.so with gcc (test infrastructure)."""
from __future__ import annotations

import os
import subprocess
import threading
import uuid

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "fff_oracle.c")
LIB = os.path.join(HERE, "libfff_oracle.so")


_lock = threading.Lock()


def build(force: bool = False) -> str:
    """Build once; safe to call from several threads or processes at the same time."""
    with _lock:
        return _build(force)


def _build(force: bool) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = LIB + f".{os.getpid()}.{uuid.uuid4().hex}.tmp"
    # -O2 without -ffast-math: summation order stays as written (k ascending).
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fPIC", "-shared",
                           "-o", tmp, SRC, "-lm"])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
