"""Compile the C oracle into two shared objects (float and double).  TEST INFRASTRUCTURE ONLY."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "sb_oracle.c")


def lib_path(real: str) -> str:
    return os.path.join(HERE, f"liboracle_{'f32' if real == 'float' else 'f64'}.so")


def build(force: bool = False) -> None:
    for real in ("float", "double"):
        out = lib_path(real)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(SRC):
            continue
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", f"-DREAL={real}",
               "-o", tmp, SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)


if __name__ == "__main__":
    build(force=True)
    print("built", lib_path("float"), lib_path("double"))
