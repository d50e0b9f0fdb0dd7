"""Per-phase times of the fused eviction kernel (diagnostic; needs the phase-stamp build of the library).

  python -m paper_2504_15364_b200.build --phase-stamps
  python -m paper_2504_15364_b200.phase_times [--workload NAME] [--steps K] [--compaction ordered]

Runs K evicting steps of the workload on the diagnostic library (every CTA's thread 0 adds the time between two
stamps to that phase's total) and prints, per phase, the mean over the CTAs of the time per unit in microseconds.
The stamps themselves cost time: use the table for proportions, the benchmark for the step time.
"""
from __future__ import annotations

import argparse
import ctypes

import numpy as np
import torch

from . import binding, build, synth

PHASES = ["prologue (first anchor)", "scores (tiles not scored earlier, register rows)", "key exchange + cluster barrier 2",
          "select + plan", "kept-index list", "evicted rows -> anchor delta", "K out / V in", "next unit's anchor",
          "V wait", "cluster barrier 3", "V out / next K in", "next unit's tiles scored", "end-of-unit barrier", "exit barrier"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama31_8b_n8192", choices=list(synth.WORKLOADS))
    ap.add_argument("--steps", type=int, default=20)
    args = ap.parse_args()
    if not build.STAMPS_LIB.exists():
        raise SystemExit("build the diagnostic library first: python -m paper_2504_15364_b200.build --phase-stamps")
    binding.LIB_PATH = build.STAMPS_LIB
    lib = binding.load_library()
    lib.keydiff_debug_phase_ns.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32]
    lib.keydiff_debug_phase_ns.restype = ctypes.c_int
    wl = synth.WORKLOADS[args.workload]
    dev = torch.device("cuda", torch.cuda.current_device())
    k_cache, v_cache, stream = synth.prefilled_cache(wl, dev)
    kd = binding.KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.budget, wl.block, path=binding.KEYDIFF_PATH_FUSED)
    kd.set_len(wl.budget)
    blocks = [stream.next_block() for _ in range(args.steps + 3)]
    for b in blocks[:3]:
        kd.evict(k_cache, v_cache, *b)
    ctas = 2368
    out = np.zeros((ctas, 16), dtype=np.uint64)
    assert lib.keydiff_debug_phase_ns(out.ctypes.data, ctas, 1) == 0   # clears the warm-up steps' totals
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for b in blocks[3:]:
        kd.evict(k_cache, v_cache, *b)
    t1.record()
    torch.cuda.synchronize()
    assert lib.keydiff_debug_phase_ns(out.ctypes.data, ctas, 0) == 0
    info = kd.launch_info()
    used = out[out.sum(1) > 0]
    per_unit = used.astype(np.float64).mean(0) * 1e-3 / args.steps / (wl.units * info["cluster_size"] / len(used))
    print(f"{wl.name}: {len(used)} CTAs, cluster size {info['cluster_size']}, {t0.elapsed_time(t1) / args.steps:.4f} ms per step (with stamps)")
    for name, us in zip(PHASES, per_unit):
        print(f"  {name:52s} {us:7.2f} us per unit")
    print(f"  {'total':52s} {per_unit.sum():7.2f} us per unit")
    kd.close()


if __name__ == "__main__":
    main()
