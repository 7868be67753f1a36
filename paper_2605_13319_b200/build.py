"""Build the CUDA library (sm_100a only) in-tree: paper_2605_13319_b200/libpipesd.so."""
from __future__ import annotations

import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libpipesd.so"
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "--use_fast_math=false"]


def _sources():
    return sorted(CSRC.glob("*.cu")) , sorted(list(CSRC.glob("*.cuh")) + [HERE.parent / "include" / "pipesd.h"])


def build_cuda(force: bool = False, verbose: bool = False) -> Path:
    cus, deps = _sources()
    newest = max(p.stat().st_mtime for p in cus + deps + [Path(__file__)])
    if not force and LIB.exists() and LIB.stat().st_mtime >= newest:
        return LIB
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    cmd = ["nvcc", *flags, *(["-Xptxas", "-v"] if verbose else []), "-o", str(LIB), *map(str, cus)]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed")
    return LIB


if __name__ == "__main__":
    build_cuda(force=True, verbose="-v" in sys.argv)
    print(LIB)
