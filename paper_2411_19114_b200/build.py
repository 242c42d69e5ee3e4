"""Builds ``libpreba.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libpreba.so"
# the same sources with -DPREBA_CHECKED: device code range-checks its offsets and addresses and
# reports a violation in the status word (PREBA_ERR_RANGE); for tests, never for measurements
LIB_CHECKED = PKG / "libpreba_checked.so"

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC,-Wall", "-shared", "-cudart", "static",
]


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu")) + sorted(CSRC.glob("*.cpp"))


def _inputs() -> list[Path]:
    return sources() + sorted(CSRC.glob("*.h")) + sorted((ROOT / "include").glob("*.h")) + [
        Path(__file__)]


def stale(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    built = lib.stat().st_mtime
    return any(p.stat().st_mtime > built for p in _inputs())


def nvcc_path() -> str:
    found = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(found):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return found


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    """Compile if the library is missing or older than its sources (``checked``: the build
    with device-side range checks)."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not stale(lib):
        return lib
    tmp = lib.with_name(f"{lib.stem}.tmp{os.getpid()}.so")
    cmd = [nvcc_path(), *NVCC_FLAGS, "-I", str(ROOT / "include"), "-I", str(CSRC)]
    if checked:
        cmd += ["-DPREBA_CHECKED"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", str(tmp)] + [str(s) for s in sources()]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv,
                checked="--checked" in sys.argv))
