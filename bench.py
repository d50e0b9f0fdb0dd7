#!/usr/bin/env python
"""Benchmark of the KeyDiff eviction step (steps/s and achieved HBM bandwidth).

A step is one ``keydiff_evict`` call over all units of the workload for one appended block, in
steady state (cache at its budget, B rows evicted per unit).  Default workload: the
Llama-3.1-8B-shaped config (32 layers x 8 KV heads, N=8192, B=128, 32K-token prompt).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--path auto|staged|fused] [--headline-only]
  python bench.py --impl reference ...        # the CPU oracle on the host cores, same metric

Prints ONE JSON line (rank 0).  Under torchrun every rank runs its own replica of the workload
(different seeded sequences); ``value`` is the whole-job rate against the slowest rank.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2504_15364_b200 import synth
from paper_2504_15364_b200 import dist as kdist

METRIC = "eviction_steps_per_s"
UNIT = "steps/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (bytes per step of the named workload); None = not captured.
NCU_TRAFFIC_BYTES = {("llama31_8b_n8192", "ordered"): 2.1161e9, ("llama31_8b_n8192", "slot_reuse"): 5.955e8,
                     ("llama32_3b_n2048", "ordered"): 4.287e8, ("llama32_3b_n2048", "slot_reuse"): 1.360e8}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, an earlier measurement of the same GPU model)"


def algorithmic_bytes(wl, moved_rows_per_step_per_unit: float, slot_reuse: bool = False) -> float:
    """Bytes one evicting step must move: every key read once, moved K rows written, moved V rows
    read and written, fp32 scores written once and read once.  With slot reuse only the kept block
    rows move (K and V, read and written), and the scores and the slot list are written once."""
    row = wl.head_dim * 2
    n = wl.budget + wl.block
    if slot_reuse:
        per_unit = n * row + 4.0 * moved_rows_per_step_per_unit * row + n * 4 + wl.budget * 4
    else:
        per_unit = n * row + 3.0 * moved_rows_per_step_per_unit * row + 2 * n * 4
    return wl.units * per_unit


class ClockSampler(threading.Thread):
    """Polls SM clock, power and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag = index, [], set(), False
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                break
            time.sleep(0.002)

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def bits(t):
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


class Run:
    """One workload on one layout, resident on the device: cache filled through the library's append path."""

    def __init__(self, wl, compaction, path, dev, rank):
        from paper_2504_15364_b200 import KeyDiff, binding
        self.wl, self.dev, self.slots = wl, dev, compaction == "slot_reuse"
        U, N, B, d = wl.units, wl.budget, wl.block, wl.head_dim
        self.stream = synth.KVStream(wl, dev, rank=rank)
        self.k_cache = torch.zeros(U, N, d, dtype=torch.bfloat16, device=dev)
        self.v_cache = torch.zeros_like(self.k_cache)
        self.kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, d, N, B, path=path, device=dev.index,
                          compaction=binding.KEYDIFF_COMPACT_SLOT_REUSE if self.slots else binding.KEYDIFF_COMPACT_ORDERED)
        self.info = self.kd.launch_info()
        self.fused = self.info["path"] == binding.KEYDIFF_PATH_FUSED
        for _ in range(wl.fill_steps):
            self.kd.evict(self.k_cache, self.v_cache, *self.stream.next_block())
        assert self.kd.len == N

    def step(self, block):
        self.kd.evict(self.k_cache, self.v_cache, *block)

    def timed(self, K, W, sampler=None):
        """W untimed steps, then K steps timed with CUDA events on the launching stream (one event pair per
        step); returns total ms, per-step ms, moved rows per unit per step."""
        blocks = [self.stream.next_block() for _ in range(W + K)]
        for i in range(W):
            self.step(blocks[i])
        torch.cuda.synchronize()
        moved0 = self.kd.moved_rows()
        st = torch.cuda.current_stream(self.dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        kdist.barrier()
        torch.cuda.synchronize()
        if sampler:
            sampler.start()
        ev[0].record(st)
        for i in range(K):
            self.step(blocks[W + i])
            ev[i + 1].record(st)
        torch.cuda.synchronize()
        if sampler:
            sampler.stop_flag = True
        kdist.barrier()
        if sampler:
            sampler.join()
        step_ms = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(K)])
        moved = (self.kd.moved_rows() - moved0) / K / self.wl.units
        status = int(self.kd.scratch()["status"].item())
        assert status == 0, f"device status {status}"
        return ev[0].elapsed_time(ev[K]), step_ms, moved

    def parity_step(self, n_units=16, cores=1, time_oracle=False):
        """One more evicting step, checked against the CPU oracle on a sample of units in this very launch
        shape.  With time_oracle the oracle is also timed on ALL units (all cores, then one thread)."""
        from oracle import compare, oracle
        wl, kd = self.wl, self.kd
        U, N = wl.units, wl.budget
        units = np.unique(np.linspace(0, U - 1, n_units).astype(int))
        sel = torch.as_tensor(units, device=self.dev)
        nk, nv = self.stream.next_block()
        timing = None
        if time_oracle:
            pre_k, pre_v = bits(self.k_cache), bits(self.v_cache)
            if self.slots:
                pos_t, next_pos = kd.positions()
                pre_pos = pos_t.cpu().numpy().astype(np.int64)

            def run_oracle(threads):
                if self.slots:
                    return oracle.evict_units_bf16_slots(pre_k, pre_v, pre_pos, N, next_pos, bits(nk), bits(nv), N, n_threads=threads)
                return oracle.evict_units_bf16(pre_k, pre_v, N, bits(nk), bits(nv), N, n_threads=threads)
            times, used = [], 1
            for rep in range(3):
                t0 = time.perf_counter()
                out = run_oracle(cores)
                times.append(time.perf_counter() - t0)
                used = out["threads"]
                if sum(times) > 12:
                    break
            t0 = time.perf_counter()
            run_oracle(1)
            single = time.perf_counter() - t0
            timing = {"value": 1.0 / float(np.mean(times)), "unit": UNIT, "cores": used, "kind": "oracle",
                      "sample": f"{len(times)} evicting step(s), all {U} units, std::thread over units",
                      "single_thread_value": 1.0 / single, "single_thread_sample": f"1 evicting step, all {U} units, 1 thread",
                      "sched_getaffinity": cores, "hardware_concurrency": os.cpu_count()}
            pre_k, pre_v = pre_k[units], pre_v[units]
            if self.slots:
                pre_pos = pre_pos[units]
        else:
            pre_k, pre_v = bits(self.k_cache[sel]), bits(self.v_cache[sel])
            if self.slots:
                pos_t, next_pos = kd.positions()
                pre_pos = pos_t[sel].cpu().numpy().astype(np.int64)
        self.step((nk, nv))
        torch.cuda.synchronize()
        sc = kd.scratch()
        scores, kept = sc["scores"][sel].cpu().numpy(), sc["kept_idx"][sel].cpu().numpy()
        if self.slots:
            rep = compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, N, bits(nk[sel]), bits(nv[sel]), N,
                                           bits(self.k_cache[sel]), bits(self.v_cache[sel]), scores, kept,
                                           kd.positions()[0][sel].cpu().numpy(), n_threads=cores)
        else:
            rep = compare.check_step(pre_k, pre_v, N, bits(nk[sel]), bits(nv[sel]), N, bits(self.k_cache[sel]),
                                     bits(self.v_cache[sel]), scores, kept, n_threads=cores)
        par = {"parity_units_checked": rep["units"], "max_score_err_over_tol": rep["max_score_err_over_tol"],
               "max_plain_rel_score_err": rep["max_plain_rel"],
               "max_plain_rel_score_err_all_tokens": rep["max_plain_rel_all_tokens"],
               "frac_tokens_with_abs_score_below_1e-2": rep["frac_tokens_below_floor"]}
        return par, timing

    def close(self):
        self.kd.close()
        del self.k_cache, self.v_cache, self.stream
        torch.cuda.empty_cache()


def roofline_of(run, moved, step_ms, workload, compaction):
    from paper_2504_15364_b200 import binding  # noqa: F401
    peak, peak_src = measured_peak()
    a_step = algorithmic_bytes(run.wl, moved, run.slots)
    kern_ms = float(step_ms.mean())
    achieved = a_step / (kern_ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": NCU_TRAFFIC_BYTES.get((workload, compaction)), "peak_source": peak_src,
            "kernel": ("slot_evict_kernel" if run.slots else "fused_evict_kernel") if run.fused else "staged chain (4 kernels)",
            "algorithmic_bytes_per_launch": a_step, "moved_rows_per_unit": moved,
            "kernel_ms": kern_ms, "kernel_ms_median": float(np.median(step_ms)),
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}


def run_ours(args):
    from paper_2504_15364_b200 import binding
    rank, world, local = kdist.init_from_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wl = synth.WORKLOADS[args.workload]
    if args.batch > 0:
        wl = synth.scaled(wl, batch=args.batch)
    if args.block > 0:
        wl = synth.scaled(wl, block=args.block)
    U, N, B, d = wl.units, wl.budget, wl.block, wl.head_dim
    path = {"auto": binding.KEYDIFF_PATH_AUTO, "staged": binding.KEYDIFF_PATH_STAGED,
            "fused": binding.KEYDIFF_PATH_FUSED}[args.path]
    K, W = args.steps, args.warmup
    K2 = 0 if args.no_e2e else 40
    cores = len(os.sched_getaffinity(0))

    run = Run(wl, args.compaction, path, dev, rank)
    info = run.info
    sampler = ClockSampler(local)
    total_ms, step_ms, moved = run.timed(K, W, sampler)
    total_ms_max = kdist.max_over_ranks(total_ms, dev)
    steps_total = kdist.sum_over_ranks(K, dev)
    value = steps_total / (total_ms_max * 1e-3)

    # ---- CPU baseline (the oracle as it stands) + a parity check in this very launch shape, taken AFTER the timed
    # steps, i.e. at the far end of the stream
    cpu = None
    if not args.no_cpu and rank == 0:
        par, cpu = run.parity_step(16, cores, time_oracle=True)
        cpu.update(par)

    # ---- end to end: block from pinned host memory, kept-index list + status read back
    e2e = None
    if K2:
        kd, stream = run.kd, run.stream
        st = torch.cuda.current_stream(dev)
        host_blocks = [tuple(t.cpu().pin_memory() for t in stream.next_block()) for _ in range(2 * K2 + 4)]
        kept_h = torch.empty(U, N, dtype=torch.int32).pin_memory()
        status_h = torch.zeros(1, dtype=torch.int32).pin_memory()
        for i in range(4):   # staging buffers, copy stream and events are created by the first call
            kd.evict_host(run.k_cache, run.v_cache, *host_blocks[i], kept_h, status_h)
        kdist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for i in range(K2):
            kd.evict_host(run.k_cache, run.v_cache, *host_blocks[4 + i], kept_h, status_h)
        e1.record(st)
        torch.cuda.synchronize()
        kdist.barrier()
        e2e_ms = kdist.max_over_ranks(e0.elapsed_time(e1), dev)
        # the same calls with the stream synchronised after every step: what a caller sees who needs the kept list
        # before it can prepare the next block (host wall clock: the wait is part of the figure)
        t0 = time.perf_counter()
        for i in range(K2):
            kd.evict_host(run.k_cache, run.v_cache, *host_blocks[4 + K2 + i], kept_h, status_h)
            st.synchronize()
        sync_ms = kdist.max_over_ranks((time.perf_counter() - t0) * 1e3, dev)
        assert int(status_h.item()) == 0
        e2e = {"value": kdist.sum_over_ranks(K2, dev) / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": 2 * U * B * d * 2, "d2h_bytes_per_step": U * N * 4 + 4, "steps": K2,
               "mode": "pipelined: calls enqueued back to back, one synchronise at the end",
               "synchronised_each_step": {"value": kdist.sum_over_ranks(K2, dev) / (sync_ms * 1e-3), "unit": UNIT,
                                          "ms_per_step": sync_ms / K2, "timer": "host wall clock, stream synchronised after every call"}}
    roof = roofline_of(run, moved, step_ms, args.workload, args.compaction) if rank == 0 else None
    run.close()

    # ---- the other workloads and the other layout, on fewer steps (rank 0 reports; every rank runs them so that
    # the ranks stay in step)
    others = []
    if not args.headline_only:
        for name in synth.CONFIG_ORDER:
            for comp in ("ordered", "slot_reuse"):
                if name == args.workload and comp == args.compaction:
                    continue
                owl = synth.WORKLOADS[name]
                r = Run(owl, comp, binding.KEYDIFF_PATH_AUTO, dev, rank)
                o_total, o_step, o_moved = r.timed(args.other_steps, 3)
                row = {"workload": name, "compaction": comp, "units": owl.units, "budget_N": owl.budget, "block_B": owl.block,
                       "path": "fused" if r.fused else "staged", "cluster_size": r.info["cluster_size"],
                       "steps": args.other_steps, "ms_per_step": kdist.max_over_ranks(o_total, dev) / args.other_steps}
                if rank == 0:
                    ro = roofline_of(r, o_moved, o_step, name, comp)
                    row.update({k: ro[k] for k in ("kernel", "algorithmic_bytes_per_launch", "achieved", "frac", "frac_of_nominal_8TBs", "traffic")})
                    if not args.no_cpu:
                        row.update(r.parity_step(16, cores)[0])
                others.append(row)
                r.close()

    if rank != 0:
        return
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "n_layers": wl.n_layers, "batch": wl.batch, "n_kv_heads": wl.n_kv_heads,
                       "head_dim": d, "budget_N": N, "block_B": B, "units": U, "key_model": wl.key_model, "storage_dtype": "bf16",
                       "cache_bytes": 2 * U * N * d * 2, "l2_policy": "inputs larger than L2 (cache >> 126 MB)",
                       "path": "fused" if info["path"] == binding.KEYDIFF_PATH_FUSED else "staged",
                       "cluster_size": info["cluster_size"], "replicas": world, "compaction": args.compaction},
            "clocks": sampler.summary(), "e2e": e2e, "gpu_launches": K * info["launches_per_step"],
            "roofline": roof, "cpu_baseline": cpu, "other_workloads": others}
    print(json.dumps(line))


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores, through its own std::thread driver over the units:
    every step scores/selects/gathers up to 256 units of the same workload; the rate is scaled to whole steps."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    wl = synth.WORKLOADS[args.workload]
    sample_units = min(wl.units, 256)
    small = wl if sample_units == wl.units else synth.scaled(wl, n_layers=1, batch=1, n_kv_heads=sample_units)
    k_cache, v_cache, stream = synth.prefilled_cache(small, "cpu")
    kc, vc = bits(k_cache), bits(v_cache)
    cores = len(os.sched_getaffinity(0))
    K, W = min(args.steps, 12), min(args.warmup, 3)
    times, used = [], 1
    for i in range(W + K):
        nk, nv = stream.next_block()
        t0 = time.perf_counter()
        out = oracle.evict_units_bf16(kc, vc, small.budget, bits(nk), bits(nv), small.budget, n_threads=cores)
        dt = time.perf_counter() - t0
        kc, vc, used = out["k"], out["v"], out["threads"]
        if i >= W:
            times.append(dt)
    per_step = float(np.mean(times)) * wl.units / sample_units
    value = 1.0 / per_step
    sample = f"{sample_units} of {wl.units} units per step, {K} steps, std::thread over units" + \
             ("" if sample_units == wl.units else ", scaled to whole steps")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
            "warmup": W, "ms_per_step": per_step * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "n_layers": wl.n_layers, "batch": wl.batch, "n_kv_heads": wl.n_kv_heads,
                       "head_dim": wl.head_dim, "budget_N": wl.budget, "block_B": wl.block, "units": wl.units,
                       "key_model": wl.key_model},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=189)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama31_8b_n8192", choices=list(synth.WORKLOADS))
    ap.add_argument("--path", default="auto", choices=["auto", "staged", "fused"])
    ap.add_argument("--compaction", default="ordered", choices=["ordered", "slot_reuse"],
                    help="layout of the kept rows: token order (the headline configuration) or unordered slot reuse")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the short runs of the other workloads and of the other layout (the other_workloads list)")
    ap.add_argument("--other-steps", type=int, default=20, help="timed steps of each entry of other_workloads")
    ap.add_argument("--batch", type=int, default=0,
                    help="run the workload at this batch size instead of its own (profiling aid: the decode workload's unit shape "
                         "at batch 2 is 2 GB instead of 34 GB); the line's config says so")
    ap.add_argument("--block", type=int, default=0,
                    help="run the workload with another block size B (0 = the workload's own), e.g. 1 for token-by-token decode")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
