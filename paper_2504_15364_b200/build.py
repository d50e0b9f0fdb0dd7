"""Build step: compile the CUDA sources in ``csrc/`` into ``libkeydiff.so`` (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libkeydiff.so"
SOURCES = [CSRC / "keydiff_api.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list((PKG.parent / "include").glob("*.h"))
    return any(p.stat().st_mtime > t for p in deps)


STAMPS_LIB = PKG / "libkeydiff_stamps.so"   # diagnostic build: fused kernel with per-phase timers (phase_times.py)
DEBUG_LIB = PKG / "libkeydiff_debug.so"     # debug build: computed row indices are range-checked into the status word


def build_library(force: bool = False, verbose: bool = False, phase_stamps: bool = False, debug_checks: bool = False) -> Path:
    """Compile libkeydiff.so in-tree if missing or older than its sources.  phase_stamps=True builds the
    diagnostic variant libkeydiff_stamps.so instead (-DKEYDIFF_PHASE_STAMPS: the fused kernel times its phases),
    debug_checks=True the variant libkeydiff_debug.so (-DKEYDIFF_DEBUG_CHECKS: row indices are range-checked)."""
    out = STAMPS_LIB if phase_stamps else DEBUG_LIB if debug_checks else LIB
    if not force and not phase_stamps and not debug_checks and not _stale():
        return out
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = out.with_suffix(f".{os.getpid()}.tmp")
    cmd = [nvcc, *NVCC_FLAGS, *(["-DKEYDIFF_PHASE_STAMPS"] if phase_stamps else []),
           *(["-DKEYDIFF_DEBUG_CHECKS"] if debug_checks else []), *(["-Xptxas", "-v"] if verbose else []),
           *map(str, SOURCES), "-o", str(tmp)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv, phase_stamps="--phase-stamps" in sys.argv,
                        debug_checks="--debug-checks" in sys.argv))
