"""Seeded random shapes through the C ABI against the CPU oracle: units, budget, block, fill level, anchor
variant, window, layout and kernel path drawn at random (all within the documented limits), two evicting
steps each."""
import numpy as np
import pytest
import torch

from oracle import compare
from paper_2504_15364_b200 import KeyDiff, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def bits(t):
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    N = int(rng.choice([7, 33, 64, 100, 257, 512, 777, 1024, 1500, 2048, 3000]))
    B = int(rng.choice([1, 3, 8, 17, 32, 64, 100, 128, 200]))
    U = int(rng.integers(1, 7))
    fill = rng.random()
    length = N if fill < 0.6 else int(rng.integers(max(0, N - B + 1), N + 1))   # full, or a transition step
    w = 0 if rng.random() < 0.5 else int(rng.integers(1, min(N, length + B) + 1))
    mode = int(rng.integers(0, 2))
    slots = bool(rng.integers(0, 2))
    path = int(rng.choice([binding.KEYDIFF_PATH_STAGED, binding.KEYDIFF_PATH_FUSED]))
    model = str(rng.choice(["offset", "outlier", "clusters", "drift"]))
    return U, N, B, length, w, mode, slots, path, model


@pytest.mark.parametrize("seed", range(48))
def test_random_configuration(seed):
    U, N, B, length, w, mode, slots, path, model = draw(seed)
    wl = synth.Workload("t", 1, 1, U, 128, N, B, model, N + 4 * B, 500 + seed)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV, length=length)
    kd = KeyDiff(1, 1, U, 128, N, max(B, 2), path=path, anchor_mode=mode, recent_window=w,
                 compaction=binding.KEYDIFF_COMPACT_SLOT_REUSE if slots else binding.KEYDIFF_COMPACT_ORDERED)
    kd.set_len(length)
    for step in range(2):
        new_k, new_v = stream.next_block(B)
        cur = kd.len
        pre_k, pre_v = bits(k_cache), bits(v_cache)
        if slots:
            pos_t, next_pos = kd.positions()
            torch.cuda.synchronize()
            pre_pos = np.tile(np.arange(N), (U, 1)) if step == 0 else pos_t.cpu().numpy().astype(np.int64)
        kd.evict(k_cache, v_cache, new_k, new_v)
        torch.cuda.synchronize()
        sc = kd.scratch()
        assert int(sc["status"].item()) == 0
        assert cur + B > N          # every drawn step evicts
        if slots:
            compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, cur, bits(new_k), bits(new_v), N, bits(k_cache), bits(v_cache),
                                     sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), kd.positions()[0].cpu().numpy(),
                                     n_threads=8, anchor_mode=mode, recent_window=w)
        else:
            compare.check_step(pre_k, pre_v, cur, bits(new_k), bits(new_v), N, bits(k_cache), bits(v_cache),
                               sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), n_threads=8,
                               anchor_mode=mode, recent_window=w)
    kd.close()


@pytest.mark.parametrize("slots", [False, True])
@pytest.mark.parametrize("seed", range(4))
def test_block_size_changes_from_step_to_step(seed, slots):
    # one context, sixteen steps with a different block size each (1 .. max_block), on the running anchor
    rng = np.random.default_rng(77 + seed)
    U, N, max_block = 3, int(rng.choice([600, 1024, 2500])), 160
    wl = synth.Workload("t", 1, 1, U, 128, N, max_block, "outlier", N + 16 * max_block, 900 + seed)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    w = int(rng.choice([0, 50]))
    kd = KeyDiff(1, 1, U, 128, N, max_block, path=binding.KEYDIFF_PATH_FUSED, recent_window=w,
                 compaction=binding.KEYDIFF_COMPACT_SLOT_REUSE if slots else binding.KEYDIFF_COMPACT_ORDERED)
    kd.set_len(N)
    worst = 0.0
    for step in range(16):
        B = int(rng.integers(1, max_block + 1))
        new_k, new_v = stream.next_block(B)
        pre_k, pre_v = bits(k_cache), bits(v_cache)
        if slots:
            pos_t, next_pos = kd.positions()
            torch.cuda.synchronize()
            pre_pos = np.tile(np.arange(N), (U, 1)) if step == 0 else pos_t.cpu().numpy().astype(np.int64)
        kd.evict(k_cache, v_cache, new_k, new_v)
        torch.cuda.synchronize()
        sc = kd.scratch()
        assert int(sc["status"].item()) == 0
        if slots:
            rep = compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, N, bits(new_k), bits(new_v), N, bits(k_cache),
                                           bits(v_cache), sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(),
                                           kd.positions()[0].cpu().numpy(), n_threads=8, recent_window=w)
        else:
            rep = compare.check_step(pre_k, pre_v, N, bits(new_k), bits(new_v), N, bits(k_cache), bits(v_cache),
                                     sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), n_threads=8, recent_window=w)
        worst = max(worst, rep["max_score_err_over_tol"])
    assert worst < 0.5
    kd.close()
