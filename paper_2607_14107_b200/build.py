"""Build the C-ABI shared library (libpolestar.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "polestar.cu")
OUT = os.path.join(HERE, "libpolestar.so")
OUT_TRACE = os.path.join(HERE, "libpolestar_trace.so")     # same library with kernel time stamps compiled in


def _deps():
    d = os.path.join(HERE, "csrc")
    files = [os.path.join(d, f) for f in os.listdir(d)]
    files.append(os.path.join(os.path.dirname(HERE), "include", "polestar.h"))
    return files


def needs_build(out: str = OUT) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(f) > t for f in _deps())


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    """Compile libpolestar.so (or, with ``trace``, libpolestar_trace.so: -DPOLESTAR_TRACE adds the
    per-kernel time stamps that `timeline.py` reads; select it with POLESTAR_LIB)."""
    out = OUT_TRACE if trace else OUT
    if not force and not needs_build(out):
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a", SRC, "-o", out]
    if trace:
        cmd.insert(1, "-DPOLESTAR_TRACE")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("nvcc failed building libpolestar.so")
    if verbose:
        sys.stderr.write(r.stderr)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, trace="--trace" in sys.argv))
