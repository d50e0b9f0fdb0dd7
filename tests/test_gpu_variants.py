"""GPU parity tests of the method's two variants against the CPU oracle, through the C ABI, on both
kernel paths: the raw-mean anchor (Sec. 3.2, text after Eq. efficient-keydiff) and KeyDiff with a
sliding window of always-kept recent tokens (Sec. 3.2)."""
import numpy as np
import pytest
import torch

from oracle import compare
from paper_2504_15364_b200 import KeyDiff, KeyDiffError, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
PATHS = [binding.KEYDIFF_PATH_STAGED, binding.KEYDIFF_PATH_FUSED]
RAW = binding.KEYDIFF_ANCHOR_RAW_MEAN


def bits(t):
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def checked_step(kd, k_cache, v_cache, new_k, new_v, mode, w, units=None):
    N, length = kd.budget, kd.len
    pre_k, pre_v = bits(k_cache), bits(v_cache)
    kd.evict(k_cache, v_cache, new_k, new_v)
    torch.cuda.synchronize()
    sc = kd.scratch()
    assert int(sc["status"].item()) == 0
    rep = compare.check_step(pre_k, pre_v, length, bits(new_k), bits(new_v), N, bits(k_cache), bits(v_cache),
                             sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(), units=units, n_threads=8,
                             anchor_mode=mode, recent_window=w)
    n = length + new_k.shape[1]
    kept = sc["kept_idx"].cpu().numpy()
    if n > N and w > 0:   # the window survives, in order, at the end of the cache
        assert (kept[:, N - w:] == np.arange(n - w, n)).all()
        assert torch.equal(k_cache[:, N - w:][:, -min(w, new_k.shape[1]):], new_k[:, -min(w, new_k.shape[1]):])
    return rep


def state(U, N, B, length, seed, model="offset"):
    wl = synth.Workload("t", 1, 1, U, 128, N, B, model, N + B, seed)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV, length=length)
    return k_cache, v_cache, stream


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode,w", [(RAW, 0), (0, 1), (0, 51), (RAW, 100), (0, 512), (RAW, 512)])
@pytest.mark.parametrize("model", ["outlier", "clusters"])
def test_single_steps(path, mode, w, model):
    U, N, B = 5, 512, 96
    k_cache, v_cache, stream = state(U, N, B, N, seed=40 + w + mode, model=model)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path, anchor_mode=mode, recent_window=w)
    kd.set_len(N)
    checked_step(kd, k_cache, v_cache, *stream.next_block(B), mode, w)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("U,N,B,length,w", [
    (3, 100, 7, 100, 10),      # ragged everything
    (2, 257, 64, 230, 26),     # transition step: len < N < len + B
    (4, 64, 200, 0, 13),       # whole prompt in one block, empty cache
    (2, 300, 1, 300, 60),      # decode cadence B = 1
    (2, 5, 3, 5, 5),           # the whole budget is window
])
def test_odd_shapes_with_window_and_raw_mean(path, U, N, B, length, w):
    for mode in (0, RAW):
        k_cache, v_cache, stream = state(U, N, B, length, seed=U * 100 + N + mode)
        kd = KeyDiff(1, 1, U, 128, N, max(B, 4), path=path, anchor_mode=mode, recent_window=w)
        kd.set_len(length)
        checked_step(kd, k_cache, v_cache, *stream.next_block(B), mode, w)
        kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode,w", [(RAW, 0), (0, 77), (RAW, 154)])
def test_streaming_with_variants(path, mode, w):
    # 10 % / 20 % of the budget as window (the paper's settings), raw-mean anchor on the running sum
    wl = synth.Workload("t", 2, 1, 3, 128, 768, 64, "outlier", 768 + 30 * 64, 61)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, 128, wl.budget, wl.block, path=path, anchor_mode=mode, recent_window=w)
    kd.set_len(wl.budget)
    worst = 0.0
    for step in range(30):
        nk, nv = stream.next_block()
        if step < 3 or step % 6 == 0 or step == 29:
            worst = max(worst, checked_step(kd, k_cache, v_cache, nk, nv, mode, w)["max_score_err_over_tol"])
        else:
            kd.evict(k_cache, v_cache, nk, nv)
    assert worst < 0.5
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_full_size_unit_with_window_and_raw_mean(path):
    # the headline unit shape (N = 8192, B = 128) on 4 units: 20 % window, raw-mean anchor
    wl = synth.scaled(synth.WORKLOADS["llama31_8b_n8192"], n_layers=1, n_kv_heads=4)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(1, 1, 4, 128, wl.budget, wl.block, path=path, anchor_mode=RAW, recent_window=1638)
    kd.set_len(wl.budget)
    for _ in range(3):
        checked_step(kd, k_cache, v_cache, *stream.next_block(), RAW, 1638)
    kd.close()


def test_bad_variant_arguments_are_rejected():
    with pytest.raises(KeyDiffError) as e:
        KeyDiff(1, 1, 2, 128, 64, 8, anchor_mode=7)
    assert e.value.code == binding.KEYDIFF_ERR_INVALID_ARG
    with pytest.raises(KeyDiffError) as e:
        KeyDiff(1, 1, 2, 128, 64, 8, recent_window=65)
    assert e.value.code == binding.KEYDIFF_ERR_INVALID_ARG
    with pytest.raises(KeyDiffError) as e:
        KeyDiff(1, 1, 2, 128, 64, 8, recent_window=-1)
    assert e.value.code == binding.KEYDIFF_ERR_INVALID_ARG


@pytest.mark.parametrize("mode,w", [(0, 0), (RAW, 900)])
def test_fused_unit_beyond_the_register_select(mode, w):
    # n = 9300 keys per unit: more than the 17 keys per thread the low-end select holds in registers,
    # so the fused kernel takes its full-table select; two steps (the second on the running anchor)
    U, N, B = 3, 9000, 300
    k_cache, v_cache, stream = state(U, N, B, N, seed=77 + w, model="outlier")
    kd = KeyDiff(1, 1, U, 128, N, B, path=binding.KEYDIFF_PATH_FUSED, anchor_mode=mode, recent_window=w)
    kd.set_len(N)
    for _ in range(2):
        checked_step(kd, k_cache, v_cache, *stream.next_block(B), mode, w)
    kd.close()


def test_fused_crowded_threshold_bin_falls_back():
    # thousands of identical keys: the threshold bin of the low-end select overflows and the kernel
    # must take the exact-rank / radix route; ties keep the older tokens
    U, N, B = 2, 2048, 128
    k_cache, v_cache, stream = state(U, N, B, N, seed=5)
    k_cache[:, 300:1900] = k_cache[:, 300:301]          # 1600 copies of one row
    new_k, new_v = stream.next_block(B)
    new_k[:, 10:90] = k_cache[:, 300:301]               # and 80 more in the block
    kd = KeyDiff(1, 1, U, 128, N, B, path=binding.KEYDIFF_PATH_FUSED)
    kd.set_len(N)
    for _ in range(2):
        checked_step(kd, k_cache, v_cache, new_k, new_v, 0, 0)
    kd.close()
