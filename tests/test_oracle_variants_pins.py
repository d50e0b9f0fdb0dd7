"""Pins for the oracle's two variants of the method, computed WITHOUT the oracle:
the raw-mean anchor (Sec. 3.2, text after Eq. efficient-keydiff: the anchor is the mean of the keys
themselves) and KeyDiff with a sliding window (Sec. 3.2: part of the budget is reserved for the most
recent tokens).  CPU only."""
import math

import numpy as np
import pytest

from oracle import oracle


def cos_to_raw_mean(K):
    """Textbook cosine of every key to the plain mean of the keys, written out in numpy."""
    K = np.asarray(K, dtype=np.float64)
    mu = K.mean(axis=0)
    return (K @ mu) / (np.linalg.norm(K, axis=1) * np.linalg.norm(mu))


def keep_with_window(e, N, w):
    """Independent restatement: the last w tokens stay; of the others the N - w with the largest e
    stay, older token first among equals.  Python sort on (-e, index) tuples."""
    n = len(e)
    if n <= N:
        return list(range(n))
    head = sorted(range(n - w), key=lambda i: (-e[i], i))[:N - w]
    return sorted(head + list(range(n - w, n)))


# ------------------------------------------------------------------ raw-mean anchor
def test_raw_mean_hand_example():
    # keys (3,0),(0,2),(-1,0),(5,5): mean (7/4, 7/4) points along (1,1); cosines 1/sqrt2, 1/sqrt2,
    # -1/sqrt2, 1 (the normalised-keys anchor gives sin/cos(pi/8) instead: the modes differ here)
    K = np.array([[3, 0], [0, 2], [-1, 0], [5, 5]], dtype=np.float64)
    out = oracle.scores(K, anchor_mode=1)
    r2 = 1 / math.sqrt(2)
    np.testing.assert_allclose(out["s"], [r2, r2, -r2, 1.0], atol=1e-15)
    np.testing.assert_allclose(out["mu"], [1.75, 1.75], atol=1e-15)
    assert abs(out["m"] - 1.75 * math.sqrt(2)) < 1e-15
    base = oracle.scores(K, anchor_mode=0)["s"]
    assert abs(base[0] - math.sin(math.pi / 8)) < 1e-12 and abs(base[3] - math.cos(math.pi / 8)) < 1e-12


@pytest.mark.parametrize("n,d,seed", [(5, 3, 0), (40, 16, 1), (300, 128, 2)])
def test_raw_mean_matches_textbook_cosine(n, d, seed):
    rng = np.random.default_rng(seed)
    K = rng.normal(size=(n, d)) * rng.uniform(0.1, 10, size=(n, 1)) + rng.normal(size=(1, d))
    np.testing.assert_allclose(oracle.scores(K, anchor_mode=1)["s"], cos_to_raw_mean(K), rtol=0, atol=1e-13)


def test_raw_mean_is_not_scale_invariant_but_normalised_is():
    rng = np.random.default_rng(3)
    K = rng.normal(size=(12, 8)) + 1.0
    K2 = K.copy()
    K2[4] *= 64.0                      # one key rescaled
    s0, s0b = oracle.scores(K)["s"], oracle.scores(K2)["s"]
    np.testing.assert_allclose(s0, s0b, atol=1e-14)                     # normalised keys: nothing changes
    s1, s1b = oracle.scores(K, anchor_mode=1)["s"], oracle.scores(K2, anchor_mode=1)["s"]
    assert np.abs(s1 - s1b).max() > 1e-3                                 # raw mean: the anchor moves
    np.testing.assert_allclose(s1b, cos_to_raw_mean(K2), atol=1e-13)


def test_modes_coincide_on_unit_keys():
    rng = np.random.default_rng(4)
    K = rng.normal(size=(30, 16))
    K /= np.linalg.norm(K, axis=1, keepdims=True)
    np.testing.assert_allclose(oracle.scores(K, anchor_mode=1)["s"], oracle.scores(K, anchor_mode=0)["s"], atol=1e-13)


def test_raw_mean_global_scale_cancels():
    rng = np.random.default_rng(5)
    K = rng.normal(size=(20, 6)) + 0.5
    np.testing.assert_allclose(oracle.scores(K * 8.0, anchor_mode=1)["s"], oracle.scores(K, anchor_mode=1)["s"], atol=1e-14)


# ------------------------------------------------------------------ sliding window
def test_window_hand_example():
    # cosines of example B (normalised anchor): sin(pi/8), cos(pi/8), -sin(pi/8), cos(pi/8); e = -cos
    c, s = math.cos(math.pi / 8), math.sin(math.pi / 8)
    e = np.array([-s, -c, s, -c])
    assert list(oracle.select(e, 3)[0]) == [0, 1, 2]                     # no window: tie 1 vs 3 keeps the older
    assert list(oracle.select(e, 3, recent_window=1)[0]) == [0, 2, 3]    # token 3 is protected, 1 is the lowest left
    assert list(oracle.select(e, 3, recent_window=2)[0]) == [0, 2, 3]    # tokens 2, 3 protected; 0 beats 1
    assert list(oracle.select(e, 3, recent_window=3)[0]) == [1, 2, 3]    # the whole budget is window
    assert list(oracle.select(e, 2, recent_window=1)[0]) == [2, 3]


@pytest.mark.parametrize("seed", range(6))
def test_window_matches_independent_definition(seed):
    rng = np.random.default_rng(100 + seed)
    for _ in range(40):
        n = int(rng.integers(2, 40))
        N = int(rng.integers(1, n + 2))
        w = int(rng.integers(0, min(N, n) + 1))
        e = np.round(rng.normal(size=n), 1)          # rounding plants ties
        S, tau = oracle.select(e, N, recent_window=w)
        want = keep_with_window(list(e), N, w)
        assert list(S) == want, (n, N, w)
        if n > N and N > w:
            head_kept = [i for i in want if i < n - w]
            assert tau == min(e[i] for i in head_kept)


def test_window_zero_is_the_plain_rule_and_full_window_keeps_the_tail():
    rng = np.random.default_rng(7)
    e = rng.normal(size=50)
    assert list(oracle.select(e, 20, recent_window=0)[0]) == list(oracle.select(e, 20)[0])
    assert list(oracle.select(e, 20, recent_window=20)[0]) == list(range(30, 50))


def test_window_all_scores_equal_keeps_oldest_plus_tail():
    e = np.zeros(12)
    assert list(oracle.select(e, 8, recent_window=3)[0]) == [0, 1, 2, 3, 4, 9, 10, 11]


# ------------------------------------------------------------------ whole step on bf16 rows
def to_bits(x):
    import torch
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def from_bits(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@pytest.mark.parametrize("mode,w", [(1, 0), (0, 5), (1, 7), (0, 16)])
def test_step_with_variants_is_scores_then_window_select_then_row_copies(mode, w):
    rng = np.random.default_rng(11 + mode + w)
    U, N, B, d, length = 3, 16, 6, 8, 16
    kc, vc = to_bits(rng.normal(size=(U, N, d)) + 0.7), to_bits(rng.normal(size=(U, N, d)))
    nk, nv = to_bits(rng.normal(size=(U, B, d)) + 0.7), to_bits(rng.normal(size=(U, B, d)))
    out = oracle.evict_units_bf16(kc, vc, length, nk, nv, N, n_threads=2, anchor_mode=mode, recent_window=w)
    for u in range(U):
        allk = np.concatenate([kc[u, :length], nk[u]]); allv = np.concatenate([vc[u, :length], nv[u]])
        K = from_bits(allk)
        if mode == 1:
            cos = cos_to_raw_mean(K)
        else:
            unit = K / np.linalg.norm(K, axis=1, keepdims=True)
            mu = unit.mean(axis=0)
            cos = (K @ mu) / (np.linalg.norm(K, axis=1) * np.linalg.norm(mu))
        np.testing.assert_allclose(out["e"][u], -cos, atol=1e-13)
        want = keep_with_window(list(out["e"][u]), N, w)
        assert list(out["S"][u]) == want
        assert (out["k"][u] == allk[want]).all() and (out["v"][u] == allv[want]).all()
        assert set(range(length + B - w, length + B)) <= set(want)
