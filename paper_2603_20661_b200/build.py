"""Build the CUDA library in-tree: nvcc, sm_100a only, one shared object."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SO = os.path.join(HERE, "libwwws.so")
SO_CHECKED = os.path.join(HERE, "libwwws_checked.so")     # -DWWWS_CHECK_INDICES: indices taken from device data are range-checked

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-Xcompiler", "-fPIC", "-shared", "--use_fast_math=false"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(SO):
        return True
    t = os.path.getmtime(SO)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(HERE, "..", "include", "wwws.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the library; `checked` builds the variant with index checks beside it
    (load it by setting WWWS_LIBRARY to its path)."""
    if not checked and not force and not needs_build():
        return SO
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [f for f in NVCC_FLAGS if f != "--use_fast_math=false"] + __import__("shlex").split(os.environ.get("WWWS_NVCC_EXTRA", ""))
    out = SO_CHECKED if checked else SO
    cmd = [nvcc] + flags + (["-DWWWS_CHECK_INDICES"] if checked else []) + (["-Xptxas", "-v"] if verbose else []) + ["-o", out] + sources()
    subprocess.check_call(cmd)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
