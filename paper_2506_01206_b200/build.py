"""Compile the CUDA library for sm_100a into ``paper_2506_01206_b200/libmdraft.so``.

nvcc cross-compiles without a GPU.  The library has a plain C ABI (see
``include/mdraft.h``) and links the CUDA runtime statically, so it can be
loaded with ctypes on a machine that has no driver (symbol checks) as well as
on the GPU machine.

Each ``csrc/*.cu`` is compiled to an object of its own (in parallel, and only
when it or a header changed) and the objects are linked into the shared
library.  ``build_library(variant="waittest")`` builds a second library,
``libmdraft_waittest.so``, for the failure-path tests: the same sources with a
short limit on every on-chip wait and an overstated byte count on every
copy barrier, so that each bounded wait runs out and the give-up paths execute.
"""

from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmdraft.so")
OBJ_DIR = os.path.join(HERE, "_build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--use_fast_math", "-Xcompiler", "-fPIC",
]

# name -> (library file, extra compile flags)
VARIANTS = {
    "": (LIB, []),
    "waittest": (os.path.join(HERE, "libmdraft_waittest.so"), ["-DMDRAFT_SPIN_LIMIT=4096u", "-DMDRAFT_TEST_OVERSTATE_TX=16u"]),
}


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h")) + [os.path.abspath(__file__)]


def _newer(deps, out: str) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(d) > t for d in deps)


def library_path(variant: str = "") -> str:
    return VARIANTS[variant][0]


def build_library(force: bool = False, verbose: bool = False, extra=(), variant: str = "") -> str:
    lib, vflags = VARIANTS[variant]
    srcs, hdrs = sources(), _headers()
    if not force and not extra and not _newer(srcs + hdrs, lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    odir = os.path.join(OBJ_DIR, variant or "main")
    os.makedirs(odir, exist_ok=True)
    flags = [*NVCC_FLAGS, *vflags, *extra]
    if verbose:
        flags = ["-Xptxas", "-v", *flags]

    def compile_one(src):
        obj = os.path.join(odir, os.path.basename(src)[:-3] + ".o")
        if force or extra or verbose or _newer([src] + hdrs, obj):
            cmd = [nvcc, *flags, "-c", "-o", obj, src]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose or r.returncode != 0:
                sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
            if r.returncode != 0:
                raise subprocess.CalledProcessError(r.returncode, cmd)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(srcs))) as pool:
        objs = list(pool.map(compile_one, srcs))
    subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib + ".tmp", *objs], check=True)
    os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    variant = "waittest" if "--waittest" in sys.argv else ""
    print(build_library(force=True, verbose="-v" in sys.argv, variant=variant))
