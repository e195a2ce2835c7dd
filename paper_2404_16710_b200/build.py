"""Build the CUDA library in-tree: ``python -m paper_2404_16710_b200.build``.

One translation unit (``csrc/ls_host.cu`` includes the kernel headers), compiled for
sm_100a only.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libls_b200.so"
TRACE_LIB = PKG / "libls_b200_trace.so"  # the same sources with -DLS_TRACE (timeline.py), never loaded by the binding

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def sources():
    return sorted(CSRC.glob("*.cu"))


def stale(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    deps = list(CSRC.glob("*")) + [ROOT / "include" / "ls.h"]
    return any(p.stat().st_mtime > t for p in deps)


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> Path:
    lib = TRACE_LIB if trace else LIB
    if not force and not stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    cmd = [nvcc, *NVCC_FLAGS, *(["-DLS_TRACE"] if trace else []), "-I", str(ROOT / "include"), "-I", str(CSRC),
           *(["-Xptxas", "-v"] if verbose else []), "-o", str(tmp), *map(str, sources())]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, trace="--trace" in sys.argv))
