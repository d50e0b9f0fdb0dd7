"""GPU parity tests: the CUDA eviction step, called through the C ABI, against the CPU oracle on
the same seeded bf16 inputs (teacher-forced, step by step).  Run with ``-m gpu`` on a B200."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import compare, oracle
from paper_2504_15364_b200 import KeyDiff, KeyDiffError, binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
PATHS = [binding.KEYDIFF_PATH_STAGED, binding.KEYDIFF_PATH_FUSED]


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def run_and_check(kd, k_cache, v_cache, new_k, new_v, units=None, n_threads=8):
    """One evicting step on the GPU, then the oracle on the pre-step state; returns the report."""
    N, length = kd.budget, kd.len
    pre_k, pre_v = bits(k_cache), bits(v_cache)
    kd.evict(k_cache, v_cache, new_k, new_v)
    torch.cuda.synchronize()
    sc = kd.scratch()
    assert int(sc["status"].item()) == 0
    rep = compare.check_step(pre_k.reshape(kd.units, N, -1), pre_v.reshape(kd.units, N, -1), length,
                             bits(new_k).reshape(kd.units, -1, kd.head_dim),
                             bits(new_v).reshape(kd.units, -1, kd.head_dim), N,
                             bits(k_cache).reshape(kd.units, N, -1), bits(v_cache).reshape(kd.units, N, -1),
                             sc["scores"].cpu().numpy(), sc["kept_idx"].cpu().numpy(),
                             units=units, n_threads=n_threads)
    # rows in front of the first evicted row must not have moved
    fe = sc["first_evicted"].cpu().numpy()
    kept = sc["kept_idx"].cpu().numpy()
    for u in (range(kd.units) if units is None else units):
        assert (kept[u, :fe[u]] == np.arange(fe[u])).all() and (fe[u] >= N or kept[u, fe[u]] > fe[u])
    return rep


def random_state(U, N, B, length, seed, model="offset"):
    wl = synth.Workload("t", 1, 1, U, 128, N, B, model, N + B, seed)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV, length=length)
    new_k, new_v = stream.next_block(B)
    return k_cache, v_cache, new_k, new_v


# ------------------------------------------------------------------------------ single steps
@pytest.mark.parametrize("path", PATHS)
def test_config1_single_step(path):
    wl = synth.WORKLOADS["single_step_n512"]
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    new_k, new_v = stream.next_block()
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.budget, wl.block, path=path)
    kd.set_len(wl.budget)
    rep = run_and_check(kd, k_cache, v_cache, new_k, new_v)
    assert rep["units"] == 8 and kd.len == 512
    kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("U,N,B,length", [
    (3, 100, 7, 100),      # ragged everything
    (1, 1000, 33, 1000),
    (5, 300, 1, 300),      # decode cadence B = 1
    (2, 257, 64, 230),     # transition step: len < N < len + B (evicts n - N < B)
    (4, 64, 200, 0),       # whole prompt in one block (B = T), empty cache
    (2, 2048, 128, 2048),
    (1, 4096, 256, 4096),
    (7, 17, 3, 17),        # tiny
    (2, 1, 1, 1),          # budget of one token
])
def test_odd_shapes(path, U, N, B, length):
    k_cache, v_cache, new_k, new_v = random_state(U, N, B, length, seed=U * 1000 + N)
    kd = KeyDiff(1, 1, U, 128, N, max(B, 4), path=path)
    kd.set_len(length)
    run_and_check(kd, k_cache, v_cache, new_k, new_v)
    assert kd.len == N
    kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("model", ["outlier", "clusters", "drift"])
def test_key_models(path, model):
    k_cache, v_cache, new_k, new_v = random_state(6, 1024, 128, 1024, seed=5, model=model)
    kd = KeyDiff(1, 1, 6, 128, 1024, 128, path=path)
    kd.set_len(1024)
    run_and_check(kd, k_cache, v_cache, new_k, new_v)
    kd.close()


# ------------------------------------------------------------------------------ paper-fixed values
@pytest.mark.parametrize("path", PATHS)
def test_hand_examples_on_gpu(path):
    # the hand-worked examples, zero-padded to 128 channels; scores against the golden cosines
    with open(os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")) as f:
        examples = json.load(f)["examples"]
    for ex in examples:
        keys = torch.tensor(ex["keys"], dtype=torch.float32)
        n = keys.shape[0]
        for N_str, want in ex["keep"].items():
            N = int(N_str)
            K = torch.zeros(1, n, 128); K[0, :, :keys.shape[1]] = keys
            V = torch.arange(n, dtype=torch.float32).view(1, n, 1).expand(1, n, 128).contiguous()
            k_cache = K[:, :N].to(torch.bfloat16).contiguous().to(DEV); v_cache = V[:, :N].to(torch.bfloat16).contiguous().to(DEV)
            new_k = K[:, N:].to(torch.bfloat16).contiguous().to(DEV); new_v = V[:, N:].to(torch.bfloat16).contiguous().to(DEV)
            kd = KeyDiff(1, 1, 1, 128, N, n - N, path=path)
            kd.set_len(N)
            kd.evict(k_cache, v_cache, new_k, new_v)
            torch.cuda.synchronize()
            sc = kd.scratch()
            np.testing.assert_allclose(-sc["scores"][0, :n].cpu().numpy(), ex["cos"], atol=2e-6)
            exact_tie = ex["name"] in ("D", "E") or ex["name"] == "A"
            if exact_tie or N_str not in ex.get("keep_if_tie_exact", {}):
                assert sc["kept_idx"][0].cpu().tolist() == want, (ex["name"], N)
                assert v_cache[0, :, 0].float().cpu().tolist() == [float(i) for i in want]
            kd.close()


# ------------------------------------------------------------------------------ degenerate inputs
@pytest.mark.parametrize("path", PATHS)
def test_all_keys_identical_keeps_oldest(path):
    U, N, B = 2, 200, 40
    row = torch.randn(1, 1, 128, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    k_cache = row.expand(U, N, 128).contiguous().to(DEV); new_k = row.expand(U, B, 128).contiguous().to(DEV)
    tag = torch.arange(N + B, dtype=torch.float32).view(1, -1, 1).expand(U, N + B, 128).to(torch.bfloat16)
    v_cache = tag[:, :N].contiguous().to(DEV); new_v = tag[:, N:].contiguous().to(DEV)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path)
    kd.set_len(N)
    run_and_check(kd, k_cache, v_cache, new_k, new_v)
    assert (kd.scratch()["kept_idx"].cpu().numpy() == np.arange(N)).all()     # ties -> oldest tokens
    assert (kd.scratch()["first_evicted"].cpu().numpy() == N).all()
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_zero_anchor_and_zero_keys(path):
    # antipodal pairs cancel the anchor exactly (all scores 0 -> index tie-break); plus zero keys
    U, N, B = 1, 64, 16
    g = torch.Generator().manual_seed(2)
    half = torch.randn(U, (N + B) // 2, 128, generator=g).to(torch.bfloat16)
    allk = torch.cat([half, -half], dim=1)
    allk[:, 5] = 0; allk[:, 5 + (N + B) // 2] = 0
    v = torch.randn(U, N + B, 128, generator=g).to(torch.bfloat16)
    k_cache, new_k = allk[:, :N].contiguous().to(DEV), allk[:, N:].contiguous().to(DEV)
    v_cache, new_v = v[:, :N].contiguous().to(DEV), v[:, N:].contiguous().to(DEV)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path)
    kd.set_len(N)
    rep = run_and_check(kd, k_cache, v_cache, new_k, new_v)
    assert rep["min_anchor_norm"] < 1e-3
    sc = kd.scratch()["scores"][0, :N + B].cpu().numpy()
    assert sc[5] == 0.0 and not np.signbit(sc[5])
    kd.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("pattern", ["first", "last", "strided", "block_only"])
def test_compaction_patterns_in_place(path, pattern):
    # Force which rows are evicted: rows to evict are copies of the dominant direction (cos ~ 1),
    # all others get a strong orthogonal component.  Exercises the in-place move hazards.
    U, N, B = 3, 1024, 128
    n = N + B
    g = torch.Generator().manual_seed(3)
    base = torch.zeros(128); base[0] = 4.0
    allk = base + torch.randn(U, n, 128, generator=g)
    evict = {"first": torch.arange(B), "last": torch.arange(N, n), "block_only": torch.arange(N, n),
             "strided": torch.arange(0, n, n // B)[:B]}[pattern]
    allk[:, evict] = base + 0.01 * torch.randn(U, len(evict), 128, generator=g)
    allk = allk.to(torch.bfloat16)
    tag = torch.randn(U, n, 128, generator=g).to(torch.bfloat16)
    k_cache, new_k = allk[:, :N].contiguous().to(DEV), allk[:, N:].contiguous().to(DEV)
    v_cache, new_v = tag[:, :N].contiguous().to(DEV), tag[:, N:].contiguous().to(DEV)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path)
    kd.set_len(N)
    run_and_check(kd, k_cache, v_cache, new_k, new_v)
    kept = kd.scratch()["kept_idx"].cpu().numpy()
    want = np.setdiff1d(np.arange(n), evict.numpy())
    assert (kept == want).all()
    kd.close()


# ------------------------------------------------------------------------------ streaming (Eq. block_processing)
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,shrink", [
    ("llama32_3b_n2048", dict(n_layers=2, budget=512, total_tokens=512 + 12 * 128)),
    ("qwen25_7b_n4096", dict(n_layers=1, batch=2, budget=768, total_tokens=768 + 6 * 256)),
    ("decode_b32_n8192", dict(n_layers=1, batch=2, budget=256, total_tokens=256 + 20 * 32)),
])
def test_block_streaming_from_empty_cache(path, name, shrink):
    wl = synth.scaled(synth.WORKLOADS[name], **shrink)
    U, N, d = wl.units, wl.budget, wl.head_dim
    stream = synth.KVStream(wl, DEV)
    k_cache = torch.zeros(U, N, d, dtype=torch.bfloat16, device=DEV); v_cache = torch.zeros_like(k_cache)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, d, N, wl.block, path=path)
    seen = 0
    while seen < wl.total_tokens:
        new_k, new_v = stream.next_block()
        if kd.len + wl.block <= N:                      # fill: append only, bit exact
            before = kd.len
            kd.evict(k_cache, v_cache, new_k, new_v)
            assert kd.len == before + wl.block
            assert torch.equal(k_cache[:, before:kd.len], new_k) and torch.equal(v_cache[:, before:kd.len], new_v)
        else:
            run_and_check(kd, k_cache, v_cache, new_k, new_v)
            assert kd.len == N
        seen += wl.block
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_tagged_values_stay_paired_and_ordered(path):
    # V rows carry the absolute token position (channel 0 = pos // 128, channel 1 = pos % 128, both
    # exact in bf16): after many steps positions must still be strictly increasing and K rows
    # must be the keys generated at those positions.
    U, N, B, T = 4, 384, 64, 384 + 64 * 10
    g = torch.Generator(device=DEV).manual_seed(4)
    keys = (1.0 + torch.randn(U, T, 128, generator=g, device=DEV)).to(torch.bfloat16)
    t = torch.arange(T, device=DEV)
    pos = torch.zeros(U, T, 128, device=DEV)
    pos[:, :, 0::2] = (t // 128).float().view(1, T, 1)
    pos[:, :, 1::2] = (t % 128).float().view(1, T, 1)
    pos = pos.to(torch.bfloat16)
    k_cache = torch.zeros(U, N, 128, dtype=torch.bfloat16, device=DEV); v_cache = torch.zeros_like(k_cache)
    kd = KeyDiff(1, 1, U, 128, N, B, path=path)
    for t0 in range(0, T, B):
        kd.evict(k_cache, v_cache, keys[:, t0:t0 + B].contiguous(), pos[:, t0:t0 + B].contiguous())
        torch.cuda.synchronize()
        L = kd.len
        assert L == min(N, t0 + B)
        p = (v_cache[:, :L, 0].float() * 128 + v_cache[:, :L, 1].float()).long()
        assert (p[:, 1:] > p[:, :-1]).all()
        assert torch.equal(v_cache[:, :L], torch.gather(pos, 1, p.unsqueeze(-1).expand(U, L, 128)))
        assert torch.equal(k_cache[:, :L], torch.gather(keys, 1, p.unsqueeze(-1).expand(U, L, 128)))
    kd.close()


# ------------------------------------------------------------------------------ full-size workloads, bench launch shape
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,sample", [("llama32_3b_n2048", 16), ("llama31_8b_n8192", 12), ("qwen25_7b_n4096", 12)])
def test_full_size_step_sampled_units(path, name, sample):
    wl = synth.WORKLOADS[name]
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.budget, wl.block, path=path)
    kd.set_len(wl.budget)
    units = np.unique(np.linspace(0, wl.units - 1, sample).astype(int))
    for step in range(2):           # a fresh-fill step, then a step on an already-evicted cache
        new_k, new_v = stream.next_block()
        run_and_check(kd, k_cache, v_cache, new_k, new_v, units=units)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_decode_config_scaled_batch(path):
    # config 5 at batch 2 (the full batch-32 cache is 34.5 GB; the kernels see the same per-unit shape)
    wl = synth.scaled(synth.WORKLOADS["decode_b32_n8192"], batch=2)
    k_cache, v_cache, stream = synth.prefilled_cache(wl, DEV)
    kd = KeyDiff(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.budget, wl.block, path=path)
    kd.set_len(wl.budget)
    units = np.unique(np.linspace(0, wl.units - 1, 10).astype(int))
    new_k, new_v = stream.next_block()
    run_and_check(kd, k_cache, v_cache, new_k, new_v, units=units)
    kd.close()


# ------------------------------------------------------------------------------ boundary behaviour
def test_errors_enqueue_nothing():
    U, N, B = 2, 64, 8
    k_cache, v_cache, new_k, new_v = random_state(U, N, B, N, seed=9)
    kd = KeyDiff(1, 1, U, 128, N, B)
    kd.set_len(N)
    before = k_cache.clone()
    big = torch.zeros(U, 2 * B, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(KeyDiffError) as ei:
        kd.evict(k_cache, v_cache, big, big.clone())               # B > max_block
    assert ei.value.code == binding.KEYDIFF_ERR_INVALID_ARG
    with pytest.raises(KeyDiffError):
        kd.evict(k_cache, v_cache, new_k[:, :, :64].contiguous(), new_v)   # wrong size
    lib = binding.load_library()
    st = torch.cuda.current_stream().cuda_stream
    args = (k_cache.data_ptr(), v_cache.data_ptr(), new_k.data_ptr(), new_v.data_ptr())
    assert lib.keydiff_evict(kd._ctx, *args, N + 1, B, U, 128, st) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_evict(kd._ctx, *args, N, B, U + 1, 128, st) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_evict(kd._ctx, *args, N, B, U, 64, st) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_evict(kd._ctx, args[0] + 2, *args[1:], N, B, U, 128, st) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_evict(kd._ctx, None, *args[1:], N, B, U, 128, st) == binding.KEYDIFF_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert kd.len == N and torch.equal(k_cache, before)
    with pytest.raises(KeyDiffError):
        kd.set_len(N + 1)
    kd.close()


@pytest.mark.parametrize("path", PATHS)
def test_deterministic_and_repeated_create_destroy(path):
    outs = []
    for rep in range(3):
        k_cache, v_cache, new_k, new_v = random_state(4, 512, 128, 512, seed=11)
        kd = KeyDiff(1, 1, 4, 128, 512, 128, path=path)
        kd.set_len(512)
        kd.evict(k_cache, v_cache, new_k, new_v)
        torch.cuda.synchronize()
        outs.append((k_cache.clone(), v_cache.clone(), kd.scratch()["scores"].clone()))
        kd.close()
    for o in outs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(outs[0], o))


@pytest.mark.parametrize("path", PATHS)
def test_host_block_entry_point(path):
    U, N, B = 4, 512, 64
    k_cache, v_cache, new_k, new_v = random_state(U, N, B, N, seed=12)
    k2, v2 = k_cache.clone(), v_cache.clone()
    kd = KeyDiff(1, 1, U, 128, N, B, path=path); kd.set_len(N)
    kd.evict(k_cache, v_cache, new_k, new_v)
    kd2 = KeyDiff(1, 1, U, 128, N, B, path=path); kd2.set_len(N)
    hk, hv = new_k.cpu().pin_memory(), new_v.cpu().pin_memory()
    kept = torch.empty(U, N, dtype=torch.int32).pin_memory(); status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    kd2.evict_host(k2, v2, hk, hv, kept, status)
    torch.cuda.synchronize()
    assert torch.equal(k_cache, k2) and torch.equal(v_cache, v2)
    assert torch.equal(kept, kd.scratch()["kept_idx"].cpu()) and int(status.item()) == 0
    kd.close(); kd2.close()


@pytest.mark.parametrize("path", PATHS)
def test_host_block_calls_back_to_back(path):
    # six calls queued without a synchronise in between: the block of one call is copied (on the ctx's copy
    # stream, into alternating staging sets) while the kernels of the call before it run; the caches must
    # end up exactly as with device-resident blocks
    wl = synth.Workload("t", 1, 1, 6, 128, 1024, 96, "outlier", 1024 + 6 * 96, 77)
    k1, v1, stream = synth.prefilled_cache(wl, DEV)
    k2, v2 = k1.clone(), v1.clone()
    blocks = [stream.next_block() for _ in range(6)]
    host = [(a.cpu().pin_memory(), b.cpu().pin_memory()) for a, b in blocks]
    kd = KeyDiff(1, 1, 6, 128, 1024, 96, path=path); kd.set_len(1024)
    kd2 = KeyDiff(1, 1, 6, 128, 1024, 96, path=path); kd2.set_len(1024)
    kept = [torch.empty(6, 1024, dtype=torch.int32).pin_memory() for _ in range(6)]
    status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    for i in range(6):
        kd2.evict_host(k2, v2, *host[i], kept[i], status)
    torch.cuda.synchronize()
    for i in range(6):
        kd.evict(k1, v1, *blocks[i])
        torch.cuda.synchronize()
        assert torch.equal(kept[i], kd.scratch()["kept_idx"].cpu()), i
    assert torch.equal(k1, k2) and torch.equal(v1, v2) and int(status.item()) == 0
    kd.close(); kd2.close()
