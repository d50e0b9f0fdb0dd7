"""Pins for the oracle's unordered slot-reuse compaction, computed WITHOUT that routine: Eq. (keydiff)
gathers the kept rows but fixes no order for them, so kept cache rows may stay where they are and the
kept block rows may take the freed slots.  Hand example, an independent Python restatement of the
placement rule, and equivalence (as a set of tokens) with the order-preserving step over a stream.
CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle


def to_bits(x):
    return torch.tensor(np.asarray(x), dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def from_bits(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def neg_cos_to_anchor(K, mode):
    """-cos(anchor, k_i) written out in numpy: anchor = mean of normalised keys (mode 0) or of the keys (1)."""
    nrm = np.linalg.norm(K, axis=1)
    mu = (K / nrm[:, None]).mean(axis=0) if mode == 0 else K.mean(axis=0)
    return -(K @ mu) / (nrm * np.linalg.norm(mu))


def place_by_definition(e, length, B, N, pos, next_pos, w):
    """The rule restated: candidates = slots 0..length-1 then block rows; tokens at the last w positions
    of the sequence stay; the others compete by (e descending, candidate number ascending) for what is
    left of N; freed slots (evicted cache rows, then empty slots) in ascending order take the kept
    block rows in block order.  Returns (src per slot, pos per slot) as lists over the valid slots."""
    n = length + B
    cand_pos = list(pos[:length]) + [next_pos + j for j in range(B)]
    if n <= N:
        return list(range(n)), cand_pos
    recent = [i for i in range(n) if cand_pos[i] >= next_pos + B - w]
    rest = [i for i in range(n) if cand_pos[i] < next_pos + B - w]
    rest_kept = sorted(rest, key=lambda i: (-e[i], i))[:max(N - len(recent), 0)]
    kept = set(recent) | set(rest_kept)
    free = [s for s in range(length) if s not in kept] + list(range(length, N))
    src = list(range(length)) + [None] * (N - length)
    newpos = list(pos[:length]) + [None] * (N - length)
    blocks = [i for i in range(length, n) if i in kept]
    assert len(blocks) == len(free)
    for s, i in zip(free, blocks):
        src[s], newpos[s] = i, cand_pos[i]
    return src, newpos


# ------------------------------------------------------------------ hand examples
HAND_K = [[1, 0], [0, 1], [1, 1], [-1, 0]]       # cache slots 0..3
HAND_B = [[1, 1], [0, -1]]                        # block rows
# unit keys sum to (sqrt2, sqrt2): the anchor points along (1,1); cosines 1/sqrt2, 1/sqrt2, 1, -1/sqrt2 | 1, -1/sqrt2


def hand_state(N):
    kc = np.zeros((1, N, 2)); kc[0, :4] = HAND_K
    vc = np.zeros((1, N, 2)); vc[0, :4] = [[10, 11], [20, 21], [30, 31], [40, 41]]
    nk = np.array([HAND_B], dtype=np.float64)
    nv = np.array([[[50, 51], [60, 61]]], dtype=np.float64)
    pos = np.zeros((1, N), dtype=np.int64); pos[0, :4] = [7, 2, 5, 0]
    return to_bits(kc), to_bits(vc), pos, to_bits(nk), to_bits(nv)


def test_hand_example_full_cache():
    # N = 4: the two keys along the anchor (slot 2 and block row 0, e = -1) go; block row 1 takes slot 2
    kc, vc, pos, nk, nv = hand_state(4)
    out = oracle.evict_units_bf16_slots(kc, vc, pos, 4, 9, nk, nv, 4)
    r2 = 1 / math.sqrt(2)
    np.testing.assert_allclose(out["e"][0], [-r2, -r2, -1, r2, -1, r2], atol=1e-15)
    assert list(out["src"][0]) == [0, 1, 5, 3]
    assert list(out["pos"][0]) == [7, 2, 10, 0]
    assert (out["k"][0] == to_bits([[1, 0], [0, 1], [0, -1], [-1, 0]])).all()
    assert (out["v"][0] == to_bits([[10, 11], [20, 21], [60, 61], [40, 41]])).all()
    assert out["len"] == 4


def test_hand_example_tie_and_empty_slot():
    # N = 5, four valid slots: one token goes; slot 2 and block row 0 tie at e = -1 and the lower
    # candidate number (the cache row) stays; block row 1 takes the empty slot 4
    kc, vc, pos, nk, nv = hand_state(5)
    out = oracle.evict_units_bf16_slots(kc, vc, pos, 4, 9, nk, nv, 5)
    assert list(out["src"][0]) == [0, 1, 2, 3, 5]
    assert list(out["pos"][0]) == [7, 2, 5, 0, 10]
    assert (out["k"][0, 4] == to_bits([0, -1])).all() and (out["v"][0, 4] == to_bits([60, 61])).all()
    assert (out["k"][0, :4] == kc[0, :4]).all()


def test_hand_example_window_on_positions():
    # window 3 with next_pos = 9: positions >= 8 are recent, i.e. both block rows (9, 10); with pos 8 planted
    # in slot 2 that slot is recent as well; two of slots 0, 1, 3 remain to be chosen for N = 4 -> 1 place:
    # slot 3 (e = +1/sqrt2) wins
    kc, vc, pos, nk, nv = hand_state(4)
    pos[0, :4] = [7, 2, 8, 0]
    out = oracle.evict_units_bf16_slots(kc, vc, pos, 4, 9, nk, nv, 4, recent_window=3)
    assert list(out["src"][0]) == [4, 5, 2, 3]          # slots 0 and 1 freed, block rows 0 and 1 placed in order
    assert list(out["pos"][0]) == [9, 10, 8, 0]


def test_append_when_the_budget_is_not_exceeded():
    kc, vc, pos, nk, nv = hand_state(8)
    out = oracle.evict_units_bf16_slots(kc, vc, pos, 4, 9, nk, nv, 8)
    assert out["e"] is None and out["len"] == 6
    assert list(out["src"][0, :6]) == [0, 1, 2, 3, 4, 5]
    assert list(out["pos"][0, :6]) == [7, 2, 5, 0, 9, 10]
    assert (out["k"][0, 4:6] == nk[0]).all() and (out["v"][0, 4:6] == nv[0]).all()


# ------------------------------------------------------------------ the rule, restated
@pytest.mark.parametrize("seed", range(8))
def test_placement_matches_independent_restatement(seed):
    rng = np.random.default_rng(200 + seed)
    for _ in range(12):
        N = int(rng.integers(3, 40)); B = int(rng.integers(1, 12)); d = 8
        length = int(rng.integers(max(0, N - B - 2), N + 1))
        w = int(rng.integers(0, min(N, length + B) + 1)) if rng.random() < 0.6 else 0
        mode = int(rng.integers(0, 2))
        base = rng.normal(size=(length + B, d)) + 0.6
        dup = rng.integers(0, length + B, size=3)           # duplicated rows plant exact ties
        base[dup] = base[dup[0]]
        kc = np.zeros((1, N, d)); kc[0, :length] = base[:length]
        vc = rng.normal(size=(1, N, d))
        nk = base[None, length:]; nv = rng.normal(size=(1, B, d))
        kcb, vcb, nkb, nvb = to_bits(kc), to_bits(vc), to_bits(nk), to_bits(nv)
        next_pos = int(rng.integers(length, length + 50))
        pos = np.zeros((1, N), dtype=np.int64); pos[0, :length] = rng.permutation(next_pos)[:length]
        out = oracle.evict_units_bf16_slots(kcb, vcb, pos, length, next_pos, nkb, nvb, N, anchor_mode=mode, recent_window=w)
        n = length + B
        allk = np.concatenate([kcb[0, :length], nkb[0]]); allv = np.concatenate([vcb[0, :length], nvb[0]])
        if n > N:
            e = out["e"][0]
            np.testing.assert_allclose(e, neg_cos_to_anchor(from_bits(allk), mode), atol=1e-13)
        else:
            e = None
        src, newpos = place_by_definition(e, length, B, N, pos[0], next_pos, w)
        valid = min(N, n)
        assert list(out["src"][0, :valid]) == src[:valid], (N, B, length, w)
        assert list(out["pos"][0, :valid]) == newpos[:valid]
        assert (out["k"][0, :valid] == allk[src[:valid]]).all() and (out["v"][0, :valid] == allv[src[:valid]]).all()


# ------------------------------------------------------------------ same tokens as the order-preserving step
@pytest.mark.parametrize("mode,w", [(0, 0), (1, 0), (0, 5), (0, 12), (1, 20)])
def test_stream_keeps_the_same_tokens_as_the_ordered_step(mode, w):
    rng = np.random.default_rng(31 + mode + w)
    U, N, B, d, steps = 2, 48, 8, 16, 25
    k_ord = to_bits(rng.normal(size=(U, N, d)) + 0.5); v_ord = to_bits(rng.normal(size=(U, N, d)))
    k_slot, v_slot = k_ord.copy(), v_ord.copy()
    pos_ord = np.tile(np.arange(N), (U, 1))
    pos_slot = pos_ord.copy()
    next_pos = N
    for _ in range(steps):
        nk = to_bits(rng.normal(size=(U, B, d)) + 0.5); nv = to_bits(rng.normal(size=(U, B, d)))
        a = oracle.evict_units_bf16(k_ord, v_ord, N, nk, nv, N, anchor_mode=mode, recent_window=w)
        b = oracle.evict_units_bf16_slots(k_slot, v_slot, pos_slot, N, next_pos, nk, nv, N, anchor_mode=mode, recent_window=w)
        for u in range(U):
            cand_pos = np.concatenate([pos_ord[u], next_pos + np.arange(B)])
            pos_ord[u] = cand_pos[a["S"][u]]
            order = np.argsort(b["pos"][u])
            assert (b["pos"][u][order] == pos_ord[u]).all()                 # the same tokens survive
            assert (b["k"][u][order] == a["k"][u]).all() and (b["v"][u][order] == a["v"][u]).all()
            changed = (b["k"][u] != k_slot[u]).any(axis=1) | (b["v"][u] != v_slot[u]).any(axis=1)
            assert changed.sum() <= B and len(set(b["pos"][u])) == N         # at most B rows move; positions distinct
            assert set(np.nonzero(b["src"][u] >= N)[0]) >= set(np.nonzero(changed)[0])
        k_ord, v_ord, k_slot, v_slot, pos_slot = a["k"], a["v"], b["k"], b["v"], b["pos"]
        next_pos += B


def test_restatement_on_hand_worked_scores():
    # the restatement itself, checked by hand on scores chosen so that a reversed block order, freed slots
    # taken from the top, or ties broken towards the block row would each give a different answer
    e = [-1.0, 0.5, -1.0, 0.7, -1.0, 0.2, 0.3]   # 4 slots + 3 block rows, N = 4: the three -1 go
    src, pos = place_by_definition(e, 4, 3, 4, [3, 2, 1, 0], 4, 0)
    assert src == [5, 1, 6, 3] and pos == [5, 2, 6, 0]   # slots 0, 2 freed; block rows 1, 2 placed in order
    e = [-1.0, 0.5, -1.0, 0.7, -1.0, 0.2]        # N = 4: two of the three -1 go, the lowest candidate number stays
    src, pos = place_by_definition(e, 4, 2, 4, [3, 2, 1, 0], 4, 0)
    assert src == [0, 1, 5, 3] and pos == [3, 2, 5, 0]
