"""GPU test of ``keydiff_evict_static``, the entry point for callers that cannot allocate device
memory (a serving process whose memory pool already owns the GPU, a plugin that is only handed
tensors).  Its scratch is a fixed array inside the library that all calls share and that keeps the
previous call's contents, so the test makes two calls in a row and compares each with the regular
``keydiff_evict`` on identical inputs: K and V must be bit-identical.

Collected last on purpose (file name), so a run that stops at the first failure has already
finished every other test.  It also passes when run alone in a fresh process.
"""
import pytest
import torch

from paper_2504_15364_b200 import KeyDiff, KeyDiffError, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _state(U, N, B, seed):
    wl = synth.Workload("t", 1, 1, U, 128, N, B, "outlier", N + 3 * B, seed)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    return k_cache, v_cache, stream


@pytest.mark.parametrize("U,N,B", [(8, 512, 128), (24, 2048, 128), (3, 1000, 33)])
def test_static_scratch_entry_matches_regular_entry_twice_in_a_row(U, N, B):
    k_ref, v_ref, stream = _state(U, N, B, seed=21)
    k_sta, v_sta = k_ref.clone(), v_ref.clone()
    kd = KeyDiff(1, 1, U, 128, N, B, path=binding.KEYDIFF_PATH_STAGED)
    kd.set_len(N)
    length = N
    for call in range(2):
        new_k, new_v = stream.next_block(B)
        kd.evict(k_ref, v_ref, new_k, new_v)
        length = binding.evict_static(k_sta, v_sta, new_k, new_v, length)
        torch.cuda.synchronize()
        assert length == N == kd.len
        assert torch.equal(k_sta, k_ref), f"call {call}: K differs"
        assert torch.equal(v_sta, v_ref), f"call {call}: V differs"
    kd.close()


def test_static_scratch_entry_appends_below_budget_and_handles_the_transition_step():
    U, N, B = 4, 300, 64
    wl = synth.Workload("t", 1, 1, U, 128, N, B, "offset", N + 4 * B, 22)
    stream = synth.KVStream(wl, DEV)
    k_ref = torch.zeros(U, N, 128, dtype=torch.bfloat16, device=DEV); v_ref = torch.zeros_like(k_ref)
    k_sta, v_sta = k_ref.clone(), v_ref.clone()
    kd = KeyDiff(1, 1, U, 128, N, B, path=binding.KEYDIFF_PATH_STAGED)
    length = 0
    for _ in range(7):     # 4 appends, the transition step (256 + 64 > 300), 2 steady steps
        new_k, new_v = stream.next_block()
        kd.evict(k_ref, v_ref, new_k, new_v)
        length = binding.evict_static(k_sta, v_sta, new_k, new_v, length)
        torch.cuda.synchronize()
        assert length == kd.len
        assert torch.equal(k_sta[:, :length], k_ref[:, :length]) and torch.equal(v_sta[:, :length], v_ref[:, :length])
    kd.close()


def test_static_scratch_entry_rejects_oversized_requests():
    # 400 units at N=8192 need ~40 MB of scratch: more than the 16 MiB array -> clear error, nothing runs
    U, N, B = 400, 8192, 128
    k = torch.zeros(U, N, 128, dtype=torch.bfloat16, device=DEV); v = torch.zeros_like(k)
    nk = torch.zeros(U, B, 128, dtype=torch.bfloat16, device=DEV); nv = torch.zeros_like(nk)
    with pytest.raises(KeyDiffError) as ei:
        binding.evict_static(k, v, nk, nv, N)
    assert ei.value.code == binding.KEYDIFF_ERR_TOO_LARGE
    assert "scratch" in str(ei.value)
    with pytest.raises(KeyDiffError) as ei:
        binding.evict_static(k, v, nk, nv, N + 1)          # len beyond the budget
    assert ei.value.code == binding.KEYDIFF_ERR_INVALID_ARG
