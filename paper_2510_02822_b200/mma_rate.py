"""Builds and runs the tensor-core rate probe (csrc/mma_rate_probe.cu): cycles per tcgen05.mma for the 8-bit
integer kind and for the narrow floating-point kind, on one SM.  Not part of the library or of any test.

    python -m paper_2510_02822_b200.mma_rate
"""
from __future__ import annotations

import os
import subprocess
import sys

from . import build as fxbuild

_DIR = os.path.dirname(os.path.abspath(__file__))


def main():
    exe = os.path.join(_DIR, "mma_rate_probe.bin")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, *[f for f in fxbuild.NVCC_FLAGS if f != "-fPIC" and f != "-Xcompiler"], os.path.join(fxbuild.CSRC, "mma_rate_probe.cu"),
           "-o", exe, "-cudart", "static"]
    subprocess.run(cmd, check=True)
    sys.exit(subprocess.run([exe]).returncode)


if __name__ == "__main__":
    main()
