"""Compile the CUDA library in-tree for sm_100a with nvcc (no GPU needed to build)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libentro.so")
LIB_CHECKED = os.path.join(HERE, "libentro_checked.so")
SOURCES = ["entro_runtime.cu", "entro_codebook.cu", "entro_quant.cu", "entro_encode.cu", "entro_decode.cu"]


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "entro.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """nvcc -> paper_2505_02380_b200/libentro.so.  Returns the library path.
    checked: the build with bounds checks on every hand-computed address (-DENTRO_CHECKED),
    libentro_checked.so beside the ordinary one; load it by setting ENTRO_LIBRARY to its path
    (pytest --checked-build does both)."""
    LIB = LIB_CHECKED if checked else globals()["LIB"]
    if not force and not _stale(LIB):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC,-ffp-contract=off",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", LIB]
    if checked:
        cmd += ["-DENTRO_CHECKED"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
