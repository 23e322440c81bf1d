"""Builds libspdp.so (the C-ABI CUDA library) in-tree for sm_100a with nvcc."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libspdp.so")
LIB_CHECKED = os.path.join(HERE, "libspdp_checked.so")      # same sources with -DSPDP_CHECKED
SOURCES = sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(HERE, "csrc", "*.h")) + glob.glob(os.path.join(HERE, "csrc", "*.cuh"))
                 + glob.glob(os.path.join(ROOT, "include", "*.h")))

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--use_fast_math=false"]


def nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def up_to_date(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(f) <= t for f in SOURCES + HEADERS + [os.path.abspath(__file__)])


def _compile(lib: str, extra, verbose: bool) -> str:
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    flags += list(extra)
    flags += os.environ.get("SPDP_NVCC_EXTRA", "").split()      # tuning hook, e.g. -DSPDP_WARPS=20
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [nvcc(), *flags, "-shared", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(HERE, "csrc"),
           "-o", tmp, *SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    return _compile(LIB, [], verbose)


def build_checked(force: bool = False) -> str:
    """The checked build: every index the kernels derive from the packed arrays is range-checked
    first and a violation lands in the device status word (see csrc/spmspv_device.cuh)."""
    if not force and up_to_date(LIB_CHECKED):
        return LIB_CHECKED
    return _compile(LIB_CHECKED, ["-DSPDP_CHECKED"], False)


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
    print(build_checked(force=True))
