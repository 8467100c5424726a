"""Builds the CUDA library in-tree: csrc/*.cu -> paper_2603_06738_b200/librib_window_attn.so.

nvcc cross-compiles for sm_100a without a GPU.  Run as ``python -m paper_2603_06738_b200.build``.
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "librib_window_attn.so"

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "-Xptxas", "-v",
]


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu"))


def stale() -> bool:
    if not LIB.exists():
        return True
    newest = max(f.stat().st_mtime for f in list(CSRC.glob("*.cu*")) + [PKG.parent / "include" / "rib_window_attn.h"])
    return LIB.stat().st_mtime < newest


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every .cu for sm_100a and link the shared library.  Raises on failure."""
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    obj_dir = PKG / "_build"
    obj_dir.mkdir(exist_ok=True)
    objs = []
    log = []
    for src in sources():
        obj = obj_dir / (src.stem + ".o")
        run = subprocess.run([nvcc, *NVCC_FLAGS, "-c", str(src), "-o", str(obj)], capture_output=True, text=True)
        log.append(run.stderr)
        if run.returncode:
            sys.stderr.write(run.stdout + run.stderr)
            raise RuntimeError(f"nvcc failed on {src.name}")
        objs.append(str(obj))
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    run = subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", *objs, "-o", str(tmp)],
                         capture_output=True, text=True)
    if run.returncode:
        sys.stderr.write(run.stdout + run.stderr)
        raise RuntimeError("link failed")
    os.replace(tmp, LIB)
    (obj_dir / "ptxas.log").write_text("\n".join(log))
    if verbose:
        print("\n".join(log))
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
