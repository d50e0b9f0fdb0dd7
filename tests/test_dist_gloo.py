"""world_size-2 gloo test (CPU) of the multi-rank plumbing the benchmark uses."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np, torch
    from paper_2504_15364_b200 import dist as kdist, synth
    rank, world, local = kdist.init_from_env("gloo")
    assert world == 2
    kdist.barrier()
    # the slowest rank sets the job time; steps add up
    assert kdist.max_over_ranks(10.0 + 5.0 * rank) == 15.0
    assert kdist.sum_over_ranks(7.0) == 14.0
    # sequences are split without overlap or loss
    mine = kdist.sequences_of_rank(5, rank, world)
    sizes = [len(kdist.sequences_of_rank(5, r, world)) for r in range(world)]
    assert sum(sizes) == 5 and list(mine) == ([0, 1, 2] if rank == 0 else [3, 4])
    # replicas draw different data per rank and identical data for the same rank
    wl = synth.scaled(synth.WORKLOADS["single_step_n512"], n_kv_heads=2, budget=32, block=8, total_tokens=40)
    a = synth.KVStream(wl, "cpu", rank=rank).next_block()[0]
    b = synth.KVStream(wl, "cpu", rank=rank).next_block()[0]
    assert torch.equal(a, b)
    digest = float(a.float().sum())
    other = [None, None]
    torch.distributed.all_gather_object(other, digest)
    assert other[0] != other[1]
    kdist.barrier()
    print("rank", rank, "ok")
""") % ROOT


def test_two_rank_gloo_plumbing(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out
