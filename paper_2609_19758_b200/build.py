"""Build the CUDA library in-tree: ``python -m paper_2609_19758_b200.build``.

Compiles every ``csrc/*.cu`` for sm_100a with nvcc into ``libfpsk.so`` next to this file.
"""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libfpsk.so")
LIB_BOUNDS = os.path.join(HERE, "libfpsk_bounds.so")       # the same sources with -DFPSK_DEBUG_BOUNDS (index checks)

def nvcc_path() -> str:
    p = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(p):
        raise RuntimeError("nvcc not found")
    return p


def sources():
    return sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(HERE, "csrc", "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(verbose: bool = False, force: bool = False, bounds: bool = False) -> str:
    """Builds libfpsk.so, or with bounds=True the index-checked variant libfpsk_bounds.so."""
    out = LIB_BOUNDS if bounds else LIB
    if not force and not needs_build(out):
        return out
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(HERE, "csrc")]
    # extra flags, e.g. FPSK_NVCC_FLAGS=-DFPSK_MEASURE for the build that records in-kernel time stamps
    cmd += os.environ.get("FPSK_NVCC_FLAGS", "").split()
    if bounds:
        cmd += ["-DFPSK_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += sources() + ["-o", out]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed")
    return out


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv, force=True, bounds="--bounds" in sys.argv))
