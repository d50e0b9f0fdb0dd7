"""B200-native KeyDiff eviction step: CUDA kernels behind a C ABI, plus a thin Python binding.

``KeyDiff`` (binding) is the public entry; ``synth`` draws the seeded synthetic workloads;
``build.build_library`` compiles the in-tree shared library.  Nothing here falls back to the CPU.
"""
from .binding import (KEYDIFF_PATH_AUTO, KEYDIFF_PATH_FUSED, KEYDIFF_PATH_STAGED, KeyDiff, KeyDiffError,
                      load_library)
from .build import build_library

__all__ = ["KeyDiff", "KeyDiffError", "load_library", "build_library",
           "KEYDIFF_PATH_AUTO", "KEYDIFF_PATH_STAGED", "KEYDIFF_PATH_FUSED"]
