"""The debug build of the library (-DKEYDIFF_DEBUG_CHECKS: every destination row index a kernel computes is
range-checked, a bad one lands in the status word as KEYDIFF_ERR_INTERNAL and the store is skipped) runs the
same steps as the product build, bit for bit, with a clean status word.  The debug library is loaded in a child
process so that this process keeps the product library."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_2504_15364_b200 import build

pytestmark = pytest.mark.gpu

CHILD = textwrap.dedent("""
    import sys, numpy as np, torch
    from paper_2504_15364_b200 import binding, build, synth
    binding.LIB_PATH = build.DEBUG_LIB if sys.argv[1] == "debug" else build.LIB
    from paper_2504_15364_b200 import KeyDiff
    out = []
    for comp, path, N, B in [(0, 2, 1536, 128), (1, 2, 1536, 128), (0, 1, 700, 33), (1, 1, 700, 33), (0, 2, 9000, 300)]:
        wl = synth.Workload("t", 1, 2, 3, 128, N, B, "outlier", N + 4 * B, 77)
        k_cache, v_cache, stream = synth.prefilled_cache(wl, "cuda")
        kd = KeyDiff(1, 2, 3, 128, N, B, path=path, compaction=comp, recent_window=40)
        kd.set_len(N)
        for _ in range(4):
            kd.evict(k_cache, v_cache, *stream.next_block())
        torch.cuda.synchronize()
        assert int(kd.scratch()["status"].item()) == 0, ("status", comp, path, N)
        out.append(int(k_cache.view(torch.int16).to(torch.int64).sum().item() * 31 + v_cache.view(torch.int16).to(torch.int64).sum().item()))
        kd.close()
    print("CHECKSUMS", out)
""")


ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run(kind):
    r = subprocess.run([sys.executable, "-c", CHILD, kind], capture_output=True, text=True, timeout=600, cwd=ROOT,
                       env={**os.environ, "PYTHONPATH": ROOT})
    assert r.returncode == 0, r.stderr[-2000:]
    return [ln for ln in r.stdout.splitlines() if ln.startswith("CHECKSUMS")][0]


def test_debug_build_runs_clean_and_matches_the_product_build():
    build.build_library()
    build.build_library(debug_checks=True)
    assert run("debug") == run("product")
