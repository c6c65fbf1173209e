"""Compile the C oracle into ``oracle/libmdraft_oracle.so`` with gcc.

Test infrastructure only: the product path never loads this library.
"""

from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "mdraft_oracle.c")
LIB = os.path.join(HERE, "libmdraft_oracle.so")


def compile_oracle(src: str = SRC, out: str = LIB, force: bool = False, extra=()) -> str:
    if (not force and os.path.exists(out)
            and os.path.getmtime(out) >= os.path.getmtime(src)):
        return out
    # -O2 without -ffast-math: fp64 arithmetic stays in the written order.
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra",
           *extra, "-o", out + ".tmp", src, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(out + ".tmp", out)
    return out


if __name__ == "__main__":
    print(compile_oracle(force="--force" in sys.argv))
