"""GPU parity tests of the unordered slot-reuse compaction against the CPU oracle, through the C ABI:
Eq. (keydiff) gathers the kept rows without fixing their order, so kept cache rows stay in their slots
and the kept block rows take the freed ones."""
import numpy as np
import pytest
import torch

from oracle import compare
from paper_2504_15364_b200 import KeyDiff, KeyDiffError, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
PATHS = [binding.KEYDIFF_PATH_STAGED, binding.KEYDIFF_PATH_FUSED]
SLOTS = binding.KEYDIFF_COMPACT_SLOT_REUSE
RAW = binding.KEYDIFF_ANCHOR_RAW_MEAN


def bits(t):
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def checked_step(kd, k_cache, v_cache, new_k, new_v, mode=0, w=0, units=None, after_set_len=False):
    """after_set_len: the ctx has just been told that slot s holds token s (it writes that down in the step)."""
    N, length = kd.budget, kd.len
    B = new_k.shape[1]
    pos_t, next_pos = kd.positions()
    torch.cuda.synchronize()
    pre_k, pre_v = bits(k_cache), bits(v_cache)
    pre_pos = np.tile(np.arange(N), (kd.units, 1)) if after_set_len else pos_t.cpu().numpy().astype(np.int64)
    moved0 = kd.moved_rows()
    kd.evict(k_cache, v_cache, new_k, new_v)
    torch.cuda.synchronize()
    sc = kd.scratch()
    assert int(sc["status"].item()) == 0
    pos_after, next_after = kd.positions()
    assert next_after == next_pos + B
    rep = compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, length, bits(new_k), bits(new_v), N,
                                   bits(k_cache), bits(v_cache), sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(),
                                   pos_after.cpu().numpy(), units=units, n_threads=8, anchor_mode=mode, recent_window=w)
    # only block rows were written: every slot that changed holds a block row now
    src = sc["kept_idx"].cpu().numpy()
    changed = (bits(k_cache) != pre_k).any(axis=2) | (bits(v_cache) != pre_v).any(axis=2)
    assert (src[changed] >= length).all()
    assert kd.moved_rows() - moved0 == int((src >= length).sum())
    return rep


def state(U, N, B, length, seed, model="offset"):
    wl = synth.Workload("t", 1, 1, U, 128, N, B, model, N + B, seed)
    return synth.prefilled_cache(wl, DEV, length=length)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode,w", [(0, 0), (RAW, 0), (0, 40), (RAW, 200)])
def test_stream_of_steps(path, mode, w):
    # 20 steps on one stream: slots fill in arbitrary order, positions follow; windows below and above B
    wl = synth.Workload("t", 2, 1, 3, 128, 640, 64, "outlier", 640 + 20 * 64, 71)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, 128, wl.budget, wl.block, path=path, anchor_mode=mode,
                 recent_window=w, compaction=SLOTS)
    kd.set_len(wl.budget)
    worst = 0.0
    for step in range(20):
        worst = max(worst, checked_step(kd, k_cache, v_cache, *stream.next_block(), mode, w,
                                        after_set_len=step == 0)["max_score_err_over_tol"])
    assert worst < 0.5
    pos, nxt = kd.positions()
    assert nxt == 640 + 20 * 64
    p = pos.cpu().numpy()
    assert all(len(set(row)) == 640 for row in p) and p.max() < nxt
    kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("U,N,B,length", [
    (3, 100, 7, 100),      # ragged everything
    (2, 257, 64, 230),     # transition step: len < N < len + B, empty slots are filled too
    (4, 64, 200, 0),       # whole prompt in one block, empty cache
    (2, 300, 1, 300),      # decode cadence B = 1
    (2, 2048, 128, 2048),
])
def test_odd_shapes(path, U, N, B, length):
    k_cache, v_cache, stream = state(U, N, B, length, seed=U * 100 + N)
    kd = KeyDiff(1, 1, U, 128, N, max(B, 4), path=path, compaction=SLOTS)
    kd.set_len(length)
    for step in range(3):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B), after_set_len=step == 0)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_prefill_from_empty_then_evict(path):
    # append-only steps fill the slots in order (positions = slots), then eviction starts
    U, N, B = 3, 256, 48
    k_cache, v_cache, stream = state(U, N, B, 0, seed=9)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path, compaction=SLOTS)
    for step in range(12):
        nk, nv = stream.next_block(B)
        if kd.len + B <= N:
            before = kd.len
            kd.evict(k_cache, v_cache, nk, nv)
            torch.cuda.synchronize()
            pos, nxt = kd.positions()
            assert nxt == before + B and (pos[:, :nxt].cpu().numpy() == np.arange(nxt)).all()
            assert torch.equal(k_cache[:, before:before + B], nk) and torch.equal(v_cache[:, before:before + B], nv)
        else:
            checked_step(kd, k_cache, v_cache, nk, nv)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_ties_keep_the_lower_candidate(path):
    U, N, B = 2, 512, 64
    k_cache, v_cache, stream = state(U, N, B, N, seed=5)
    k_cache[:, 100:400] = k_cache[:, 100:101]          # 300 copies of one row
    new_k, new_v = stream.next_block(B)
    new_k[:, 10:40] = k_cache[:, 100:101]
    kd = KeyDiff(1, 1, U, 128, N, B, path=path, compaction=SLOTS)
    kd.set_len(N)
    for step in range(2):
        checked_step(kd, k_cache, v_cache, new_k, new_v, after_set_len=step == 0)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_full_size_unit(path):
    wl = synth.scaled(synth.WORKLOADS["llama31_8b_n8192"], n_layers=1, n_kv_heads=4)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(1, 1, 4, 128, wl.budget, wl.block, path=path, compaction=SLOTS, recent_window=819)
    kd.set_len(wl.budget)
    for step in range(3):
        checked_step(kd, k_cache, v_cache, *stream.next_block(), 0, 819, after_set_len=step == 0)
    kd.close()


def test_same_tokens_survive_as_in_the_ordered_layout():
    # two contexts on the same stream, one per layout: after every step the slot cache, sorted by
    # position, holds the rows of the ordered cache (scores differ only in summation order, so a flip
    # needs a near-tie at the threshold: not with these seeds)
    wl = synth.Workload("t", 1, 1, 4, 128, 512, 32, "outlier", 512 + 15 * 32, 13)
    k1, v1, stream = synth.prefilled_cache(wl, DEV)
    k2, v2 = k1.clone(), v1.clone()
    a = KeyDiff(1, 1, 4, 128, 512, 32, path=binding.KEYDIFF_PATH_STAGED)
    b = KeyDiff(1, 1, 4, 128, 512, 32, path=binding.KEYDIFF_PATH_STAGED, compaction=SLOTS)
    a.set_len(512); b.set_len(512)
    for _ in range(15):
        nk, nv = stream.next_block()
        a.evict(k1, v1, nk, nv); b.evict(k2, v2, nk, nv)
        torch.cuda.synchronize()
        order = torch.argsort(b.positions()[0].long(), dim=1)
        idx = order[:, :, None].expand(-1, -1, 128)
        assert torch.equal(torch.gather(k2, 1, idx), k1) and torch.equal(torch.gather(v2, 1, idx), v1)
    a.close(); b.close()


def test_positions_need_the_slot_layout_and_bad_values_are_rejected():
    kd = KeyDiff(1, 1, 2, 128, 64, 8)
    with pytest.raises(KeyDiffError) as e:
        kd.positions()
    assert e.value.code == binding.KEYDIFF_ERR_STATE
    kd.close()
    with pytest.raises(KeyDiffError) as e:
        KeyDiff(1, 1, 2, 128, 64, 8, compaction=3)
    assert e.value.code == binding.KEYDIFF_ERR_INVALID_ARG


@pytest.mark.parametrize("path", PATHS)
def test_rebuilding_the_anchor_every_step_and_reset(path):
    # set_incremental(False): the running sum is rebuilt from the cache rows before every step; reset starts a
    # new sequence (positions from 0 again); both give oracle-exact steps
    U, N, B = 3, 384, 32
    k_cache, v_cache, stream = state(U, N, B, N, seed=21, model="outlier")
    kd = KeyDiff(1, 1, U, 128, N, B, path=path, compaction=SLOTS)
    kd.set_incremental(False)
    kd.set_len(N)
    for step in range(4):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B), after_set_len=step == 0)
    kd.set_incremental(True)
    for step in range(3):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B))
    kd.reset()
    assert kd.len == 0 and kd.positions()[1] == 0
    for step in range(N // B):
        kd.evict(k_cache, v_cache, *stream.next_block(B))
    assert kd.len == N
    for step in range(3):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B))
    kd.close()


def test_block_from_host_memory():
    # keydiff_evict_host with slot reuse: the slot list read back is the one in scratch
    U, N, B = 4, 512, 64
    k_cache, v_cache, stream = state(U, N, B, N, seed=33)
    kd = KeyDiff(1, 1, U, 128, N, B, compaction=SLOTS)
    kd.set_len(N)
    kept_h = torch.empty(U, N, dtype=torch.int32).pin_memory()
    status_h = torch.ones(1, dtype=torch.int32).pin_memory()
    for step in range(3):
        nk, nv = stream.next_block(B)
        pre_k, pre_v = bits(k_cache), bits(v_cache)
        pre_pos = np.tile(np.arange(N), (U, 1)) if step == 0 else kd.positions()[0].cpu().numpy().astype(np.int64)
        next_pos = kd.positions()[1]
        kd.evict_host(k_cache, v_cache, nk.cpu().pin_memory(), nv.cpu().pin_memory(), kept_h, status_h)
        torch.cuda.synchronize()
        assert int(status_h.item()) == 0
        sc = kd.scratch()
        assert torch.equal(kept_h, sc["kept_idx"].cpu())
        compare.check_step_slots(pre_k, pre_v, pre_pos, next_pos, N, bits(nk), bits(nv), N, bits(k_cache), bits(v_cache),
                                 sc["scores"].cpu().numpy(), kept_h.numpy(), kd.positions()[0].cpu().numpy(), n_threads=8)
    kd.close()


def test_decode_cadence_one_token_per_step():
    # B = 1 at the headline unit shape: every step scores 8193 keys and replaces one slot
    wl = synth.scaled(synth.WORKLOADS["llama31_8b_n8192"], n_layers=1, n_kv_heads=3, block=1)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(1, 1, 3, 128, wl.budget, 1, compaction=SLOTS)
    kd.set_len(wl.budget)
    for step in range(6):
        nk, nv = stream.next_block(1)
        if step in (0, 1, 5):
            checked_step(kd, k_cache, v_cache, nk, nv, after_set_len=step == 0)
        else:
            kd.evict(k_cache, v_cache, nk, nv)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_all_keys_identical_nothing_is_written(path):
    # every score ties: the lower candidate numbers (the cache slots) stay, every block row goes, no slot changes
    U, N, B = 2, 200, 40
    row = torch.randn(1, 1, 128, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    k_cache = row.expand(U, N, 128).contiguous().to(DEV); new_k = row.expand(U, B, 128).contiguous().to(DEV)
    tag = torch.arange(N + B, dtype=torch.float32).view(1, -1, 1).expand(U, N + B, 128).to(torch.bfloat16)
    v_cache = tag[:, :N].contiguous().to(DEV); new_v = tag[:, N:].contiguous().to(DEV)
    before_k, before_v = k_cache.clone(), v_cache.clone()
    kd = KeyDiff(1, 1, U, 128, N, B, path=path, compaction=SLOTS)
    kd.set_len(N)
    checked_step(kd, k_cache, v_cache, new_k, new_v, after_set_len=True)
    assert (kd.scratch()["kept_idx"].cpu().numpy() == np.arange(N)).all()
    assert torch.equal(k_cache, before_k) and torch.equal(v_cache, before_v)
    assert (kd.positions()[0].cpu().numpy() == np.arange(N)).all() and kd.positions()[1] == N + B
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_zero_anchor_and_zero_keys(path):
    # antipodal pairs cancel the anchor exactly (all scores 0 -> candidate-number tie-break); plus zero keys
    U, N, B = 1, 64, 16
    g = torch.Generator().manual_seed(2)
    half = torch.randn(U, (N + B) // 2, 128, generator=g).to(torch.bfloat16)
    allk = torch.cat([half, -half], dim=1)
    allk[:, 5] = 0; allk[:, 5 + (N + B) // 2] = 0
    v = torch.randn(U, N + B, 128, generator=g).to(torch.bfloat16)
    k_cache, new_k = allk[:, :N].contiguous().to(DEV), allk[:, N:].contiguous().to(DEV)
    v_cache, new_v = v[:, :N].contiguous().to(DEV), v[:, N:].contiguous().to(DEV)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path, compaction=SLOTS)
    kd.set_len(N)
    rep = checked_step(kd, k_cache, v_cache, new_k, new_v, after_set_len=True)
    assert rep["min_anchor_norm"] < 1e-3
    sc = kd.scratch()["scores"][0, :N + B].cpu().numpy()
    assert sc[5] == 0.0 and not np.signbit(sc[5])
    kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("model", ["clusters", "drift"])
def test_key_models(path, model):
    wl = synth.Workload("t", 1, 2, 3, 128, 1024, 128, model, 1024 + 8 * 128, 91)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, 128, wl.budget, wl.block, path=path, compaction=SLOTS)
    kd.set_len(wl.budget)
    for step in range(8):
        checked_step(kd, k_cache, v_cache, *stream.next_block(), after_set_len=step == 0)
    kd.close()


def test_blocks_beyond_the_streaming_kernel_go_to_the_staged_path():
    # the streaming kernel keeps three max_block-sized lists in shared memory and is built for max_block <= 1024
    U, N, B = 2, 2048, 1500
    with pytest.raises(KeyDiffError) as e:
        KeyDiff(1, 1, U, 128, N, B, path=binding.KEYDIFF_PATH_FUSED, compaction=SLOTS)
    assert e.value.code == binding.KEYDIFF_ERR_UNSUPPORTED
    kd = KeyDiff(1, 1, U, 128, N, B, compaction=SLOTS)
    assert kd.launch_info()["path"] == binding.KEYDIFF_PATH_STAGED
    k_cache, v_cache, stream = state(U, N, B, N, seed=3)
    kd.set_len(N)
    for step in range(2):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B), after_set_len=step == 0)
    kd.close()


@pytest.mark.parametrize("U,N,B,w", [(3, 9000, 300, 0), (3, 9000, 300, 900), (2, 17000, 400, 0)])
def test_units_beyond_the_register_select(U, N, B, w):
    # more than 17 keys per thread: the streaming kernel takes the full-table select, which fills the same
    # bitmap; beyond 16384 candidates the bitmap's prefix runs over more than one 512-word chunk
    k_cache, v_cache, stream = state(U, N, B, N, seed=70 + w, model="outlier")
    kd = KeyDiff(1, 1, U, 128, N, B, path=binding.KEYDIFF_PATH_FUSED, compaction=SLOTS, recent_window=w)
    kd.set_len(N)
    for step in range(2):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B), 0, w, after_set_len=step == 0)
    kd.close()
