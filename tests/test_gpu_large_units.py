"""GPU parity for units beyond 8704 keys, where the low-end selection reads its keys from the shared-memory table
instead of registers: a 16K budget on both layouts (the ordered layout then runs on the staged kernels, slot reuse
on the streaming kernel), an 8K budget with a 640-token block on the fused cluster kernel, and heavy ties."""
import numpy as np
import pytest
import torch

from oracle import compare
from paper_2504_15364_b200 import KeyDiff, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def bits(t):
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def run_steps(wl, compaction, steps, path=binding.KEYDIFF_PATH_AUTO, window=0):
    N = wl.budget
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, N, wl.block, path=path, compaction=compaction,
                 recent_window=window)
    kd.set_len(N)
    slots = compaction == binding.KEYDIFF_COMPACT_SLOT_REUSE
    info = kd.launch_info()
    for step in range(steps):
        nk, nv = stream.next_block()
        pre_k, pre_v = bits(k_cache), bits(v_cache)
        if slots:
            pos_t, next_pos = kd.positions()
            torch.cuda.synchronize()
            pre_pos = np.tile(np.arange(N), (wl.units, 1)) if step == 0 else pos_t.cpu().numpy().astype(np.int64)
        kd.evict(k_cache, v_cache, nk, nv)
        torch.cuda.synchronize()
        sc = kd.scratch()
        assert int(sc["status"].item()) == 0
        if slots:
            compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, N, bits(nk), bits(nv), N, bits(k_cache), bits(v_cache),
                                     sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), kd.positions()[0].cpu().numpy(),
                                     n_threads=8, recent_window=window)
        else:
            compare.check_step(pre_k, pre_v, N, bits(nk), bits(nv), N, bits(k_cache), bits(v_cache),
                               sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), n_threads=8, recent_window=window)
    kd.close()
    return info


@pytest.mark.parametrize("compaction", [binding.KEYDIFF_COMPACT_ORDERED, binding.KEYDIFF_COMPACT_SLOT_REUSE])
def test_budget_16384_block_128(compaction):
    wl = synth.Workload("t", 1, 1, 4, 128, 16384, 128, "outlier", 16384 + 4 * 128, 41)
    info = run_steps(wl, compaction, 3)
    if compaction == binding.KEYDIFF_COMPACT_SLOT_REUSE:
        assert info["path"] == binding.KEYDIFF_PATH_FUSED      # the streaming kernel, selection over 16512 keys


@pytest.mark.parametrize("window", [0, 500])
def test_budget_8192_block_640_on_the_cluster_kernel(window):
    wl = synth.Workload("t", 1, 1, 3, 128, 8192, 640, "drift", 8192 + 4 * 640, 42)
    info = run_steps(wl, binding.KEYDIFF_COMPACT_ORDERED, 3, path=binding.KEYDIFF_PATH_FUSED, window=window)
    assert info["path"] == binding.KEYDIFF_PATH_FUSED


@pytest.mark.parametrize("compaction", [binding.KEYDIFF_COMPACT_ORDERED, binding.KEYDIFF_COMPACT_SLOT_REUSE])
def test_many_equal_scores_beyond_8704_keys(compaction):
    # every key is one of three directions: thousands of exactly equal scores, the threshold bin is crowded and the
    # selection must take the full-table route and still keep the oldest tokens among equals
    N, B, U = 9000, 300, 2
    g = torch.Generator(device="cpu").manual_seed(7)
    dirs = torch.randn(3, 128, generator=g)
    pick = torch.randint(0, 3, (U, N + 2 * B), generator=g)
    scale = torch.tensor([1.0, 2.0, 4.0])[torch.randint(0, 3, (U, N + 2 * B), generator=g)]
    allk = (dirs[pick] * scale.unsqueeze(-1)).to(torch.bfloat16).to(DEV)
    allv = torch.randn(U, N + 2 * B, 128, generator=g).to(torch.bfloat16).to(DEV)
    k_cache, v_cache = allk[:, :N].contiguous(), allv[:, :N].contiguous()
    kd = KeyDiff(1, 1, U, 128, N, B, compaction=compaction)
    kd.set_len(N)
    slots = compaction == binding.KEYDIFF_COMPACT_SLOT_REUSE
    for step in range(2):
        nk, nv = allk[:, N + step * B:N + (step + 1) * B].contiguous(), allv[:, N + step * B:N + (step + 1) * B].contiguous()
        pre_k, pre_v = bits(k_cache), bits(v_cache)
        if slots:
            pos_t, next_pos = kd.positions()
            torch.cuda.synchronize()
            pre_pos = np.tile(np.arange(N), (U, 1)) if step == 0 else pos_t.cpu().numpy().astype(np.int64)
        kd.evict(k_cache, v_cache, nk, nv)
        torch.cuda.synchronize()
        sc = kd.scratch()
        assert int(sc["status"].item()) == 0
        if slots:
            compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, N, bits(nk), bits(nv), N, bits(k_cache), bits(v_cache),
                                     sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), kd.positions()[0].cpu().numpy(), n_threads=8)
        else:
            compare.check_step(pre_k, pre_v, N, bits(nk), bits(nv), N, bits(k_cache), bits(v_cache),
                               sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), n_threads=8)
    kd.close()
