"""Build the CUDA shared library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libadwin_b200.so"
LIB_CHECKED = PKG / "libadwin_b200_checked.so"   # -DADWIN_CHECKED: every hand-made index tested

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def sources():
    return sorted(CSRC.glob("*.cu"))


def needs_build(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    newest = max(p.stat().st_mtime for p in list(CSRC.iterdir()) + [PKG.parent / "include" / "adwin.h"])
    return lib.stat().st_mtime < newest


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    """Build the library (or, with checked=True, its bounds-checked flavour, which stands in for a
    memory checker: every shared-memory / ring / record / global index the kernels form is tested,
    a violation skips the access and raises ADWIN_DEV_BOUNDS; same exports, slower kernels)."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not needs_build(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib.with_suffix(f".tmp{os.getpid()}.so")
    cmd = [nvcc, *NVCC_FLAGS, *(["-DADWIN_CHECKED"] if checked else []),
           *(["-Xptxas", "-v"] if verbose else []), *[str(s) for s in sources()], "-o", str(tmp)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError(f"nvcc failed building {lib.name}")
    if verbose:
        print(res.stderr)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv,
                checked="--checked" in sys.argv))
