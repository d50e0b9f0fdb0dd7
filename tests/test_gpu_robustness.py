"""GPU tests of the library's failure handling and state hand-over: a bounded device wait that runs out,
allocation failure inside keydiff_create, and resuming a slot-reuse cache from saved positions.  Nothing here
faults, traps or hangs the device: the wait that runs out is a wait on a barrier nothing completes, with a
limit of a thousand polls, after which the kernel returns by itself."""
import numpy as np
import pytest
import torch

from oracle import compare
from paper_2504_15364_b200 import KeyDiff, KeyDiffError, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def bits(t):
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def test_a_bounded_wait_that_runs_out_reports_timeout_and_the_context_stays_usable():
    assert binding.selftest_bounded_wait(1000) == binding.KEYDIFF_ERR_TIMEOUT
    assert binding.selftest_bounded_wait(1) == binding.KEYDIFF_ERR_TIMEOUT
    # the device is as usable as before: an ordinary step right after it is correct
    wl = synth.WORKLOADS["single_step_n512"]
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    nk, nv = stream.next_block()
    pre_k, pre_v = bits(k_cache), bits(v_cache)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.budget, wl.block)
    kd.set_len(wl.budget)
    kd.evict(k_cache, v_cache, nk, nv)
    torch.cuda.synchronize()
    sc = kd.scratch()
    assert int(sc["status"].item()) == 0
    compare.check_step(pre_k, pre_v, wl.budget, bits(nk), bits(nv), wl.budget, bits(k_cache), bits(v_cache),
                       sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy())
    kd.close()
    lib = binding.load_library()
    assert lib.keydiff_selftest_bounded_wait(None, 1000, None) == binding.KEYDIFF_ERR_INVALID_ARG
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert lib.keydiff_selftest_bounded_wait(status.data_ptr(), 0, None) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_selftest_bounded_wait(status.data_ptr(), 1 << 20, None) == binding.KEYDIFF_ERR_INVALID_ARG


@pytest.mark.parametrize("compaction", [binding.KEYDIFF_COMPACT_ORDERED, binding.KEYDIFF_COMPACT_SLOT_REUSE])
def test_allocation_failure_in_create_releases_everything(compaction):
    torch.cuda.synchronize()
    args = dict(path=binding.KEYDIFF_PATH_AUTO, compaction=compaction)
    KeyDiff(2, 1, 4, 128, 1024, 64, **args).close()          # warm: module loading, attributes
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    failures = 0
    for nth in range(1, 16):
        binding.debug_fail_alloc(nth)
        try:
            kd = KeyDiff(2, 1, 4, 128, 1024, 64, **args)
        except KeyDiffError as e:
            assert e.code == binding.KEYDIFF_ERR_ALLOC
            failures += 1
            continue
        kd.close()        # nth is past the last allocation of create: the hook was disarmed by create's return
        break
    assert failures >= 10, failures          # every allocation of keydiff_create was made to fail once
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free0 - (2 << 20), "a failed keydiff_create leaked device memory"
    kd = KeyDiff(2, 1, 4, 128, 1024, 64, **args)            # and the library still works
    kd.close()


def run_slot_stream(wl, window, steps, incremental, resume_at=None):
    """Slot-reuse stream of `steps` evicting steps; with resume_at = s the caches, positions and next position
    are saved after step s, the ctx is destroyed, and a NEW ctx continues from the saved state."""
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    mk = lambda: KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.budget, wl.block, recent_window=window,
                         compaction=binding.KEYDIFF_COMPACT_SLOT_REUSE)
    kd = mk()
    kd.set_incremental(incremental)
    kd.set_len(wl.budget)
    for s in range(steps):
        if resume_at is not None and s == resume_at:
            torch.cuda.synchronize()
            pos_t, next_pos = kd.positions()
            saved = (k_cache.clone(), v_cache.clone(), pos_t.clone(), next_pos, kd.len)
            kd.close()
            k_cache, v_cache = saved[0], saved[1]
            kd = mk()
            kd.set_incremental(incremental)
            kd.set_positions(saved[2], saved[4], saved[3])
        kd.evict(k_cache, v_cache, *stream.next_block())
    torch.cuda.synchronize()
    out = (k_cache.clone(), v_cache.clone(), kd.positions()[0].clone(), kd.positions()[1])
    kd.close()
    return out


@pytest.mark.parametrize("window", [0, 96])
def test_slot_reuse_cache_resumes_from_saved_positions_bit_for_bit(window):
    # both runs rebuild the anchor from all rows every step, so that they perform the same arithmetic
    # (a resumed ctx has to rebuild it anyway) and the comparison can be exact
    wl = synth.Workload("t", 1, 2, 3, 128, 768, 64, "outlier", 768 + 20 * 64, 31)
    ref = run_slot_stream(wl, window, 20, incremental=False)
    got = run_slot_stream(wl, window, 20, incremental=False, resume_at=10)
    assert torch.equal(ref[0], got[0]) and torch.equal(ref[1], got[1])
    assert torch.equal(ref[2], got[2]) and ref[3] == got[3]
    assert not torch.equal(ref[2][0], torch.arange(768, dtype=torch.int32, device=DEV)), "the stream never reused a slot"


def test_resumed_slot_reuse_cache_on_the_running_anchor_matches_the_oracle():
    wl = synth.Workload("t", 1, 1, 4, 128, 1024, 128, "drift", 1024 + 12 * 128, 32)
    N = wl.budget
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    mk = lambda: KeyDiff(1, 1, 4, 128, N, 128, recent_window=100, compaction=binding.KEYDIFF_COMPACT_SLOT_REUSE)
    kd = mk()
    kd.set_len(N)
    for _ in range(6):
        kd.evict(k_cache, v_cache, *stream.next_block())
    torch.cuda.synchronize()
    pos_saved, next_pos = kd.positions()
    pos_saved = pos_saved.clone()
    kd.close()
    kd = mk()
    kd.set_positions(pos_saved, N, next_pos)
    assert torch.equal(kd.positions()[0], pos_saved) and kd.positions()[1] == next_pos and kd.len == N
    for _ in range(6):
        nk, nv = stream.next_block()
        pre_k, pre_v = bits(k_cache), bits(v_cache)
        pos_t, nxt = kd.positions()
        pre_pos = pos_t.cpu().numpy().astype(np.int64)
        kd.evict(k_cache, v_cache, nk, nv)
        torch.cuda.synchronize()
        sc = kd.scratch()
        compare.check_step_slots(pre_k, pre_v, pre_pos, nxt, N, bits(nk), bits(nv), N, bits(k_cache), bits(v_cache),
                                 sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), kd.positions()[0].cpu().numpy(),
                                 recent_window=100)
    kd.close()


def test_set_positions_identity_and_argument_checks():
    kd = KeyDiff(1, 1, 2, 128, 256, 32, compaction=binding.KEYDIFF_COMPACT_SLOT_REUSE)
    kd.set_positions(None, 200, 200)
    torch.cuda.synchronize()
    assert torch.equal(kd.positions()[0][0], torch.arange(256, dtype=torch.int32, device=DEV)) and kd.len == 200
    with pytest.raises(KeyDiffError) as e:
        kd.set_positions(None, 300, 300)          # len > budget
    assert e.value.code == binding.KEYDIFF_ERR_INVALID_ARG
    with pytest.raises(KeyDiffError) as e:
        kd.set_positions(None, 100, 50)           # next position below the length
    assert e.value.code == binding.KEYDIFF_ERR_INVALID_ARG
    kd.close()
    kd = KeyDiff(1, 1, 2, 128, 256, 32)           # ordered layout: no positions
    with pytest.raises(KeyDiffError) as e:
        kd.set_positions(None, 10, 10)
    assert e.value.code == binding.KEYDIFF_ERR_STATE
    kd.close()
