"""Pins for the CPU oracle (no GPU).

Each test checks the oracle against something fixed by the paper or by mathematics
and computed WITHOUT the oracle: hand-derived closed forms (tests/golden), the
pairwise definition Eq. (keydiff) evaluated with numpy, exhaustive enumeration of
subsets for the relaxed objective Eq. (relaxed_min_cossim_opt), and structural
invariants of Eq. (eviction_policy) / Eq. (block_processing).
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")
with open(GOLDEN) as f:
    EXAMPLES = {e["name"]: e for e in json.load(f)["examples"]}


def bf16_bits(x):
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- hand-worked examples
@pytest.mark.parametrize("name", sorted(EXAMPLES))
def test_hand_example_scores(name):
    ex = EXAMPLES[name]
    out = oracle.scores(np.array(ex["keys"], dtype=np.float64))
    np.testing.assert_allclose(out["s"], ex["cos"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(out["mu"], ex["mu"], rtol=0, atol=1e-15)
    if "m" in ex:
        assert abs(out["m"] - ex["m"]) < 1e-15


@pytest.mark.parametrize("name", sorted(EXAMPLES))
def test_hand_example_selection(name):
    ex = EXAMPLES[name]
    s = oracle.scores(np.array(ex["keys"], dtype=np.float64))["s"]
    e = oracle.eviction_scores(s)
    for N, want in ex["keep"].items():
        S, tau = oracle.select(e, int(N))
        assert S.tolist() == want, (name, N)
        assert tau == min(e[S])
    # where two tokens tie exactly in real arithmetic, floating point may separate them
    # by an ulp: feeding the exact golden cosines must give the tie-break result.
    for N, want in ex.get("keep_if_tie_exact", {}).items():
        S, _ = oracle.select(oracle.eviction_scores(np.array(ex["cos"])), int(N))
        assert S.tolist() == want


def test_example_b_distinguishes_normalised_from_raw_anchor():
    # With the mean of the RAW keys as anchor the cosines of example B would be
    # (.7071, .7071, -.7071, 1); the oracle must give the normalised-anchor values.
    ex = EXAMPLES["B"]
    s = oracle.scores(np.array(ex["keys"], dtype=np.float64))["s"]
    assert np.max(np.abs(s - np.array(ex["raw_mean_cos"]))) > 0.07
    # and positive rescaling of single keys changes nothing
    s2 = oracle.scores(np.array(ex["rescaled_keys"], dtype=np.float64))["s"]
    np.testing.assert_allclose(s2, ex["cos"], atol=1e-14)


def test_hand_example_through_bf16_head_routine():
    # Example C has small-integer keys (exact in bf16).  N=2 keeps tokens 0 and 3 and the
    # compacted rows must come out in token order, with V following K.
    ex = EXAMPLES["C"]
    keys = np.array(ex["keys"], dtype=np.float32)
    vals = np.arange(12, dtype=np.float32).reshape(4, 3) + 100
    N = 2
    kc = np.zeros((1, N, 3), np.uint16); vc = np.zeros((1, N, 3), np.uint16)
    kc[0] = bf16_bits(keys[:2]); vc[0] = bf16_bits(vals[:2])
    out = oracle.evict_units_bf16(kc, vc, 2, bf16_bits(keys[2:])[None], bf16_bits(vals[2:])[None], N)
    assert out["S"].tolist() == [[0, 3]]
    np.testing.assert_allclose(-out["e"][0], ex["cos"], atol=1e-14)
    assert abs(out["m"][0] - ex["m"]) < 1e-15
    assert (out["k"][0] == bf16_bits(keys[[0, 3]])).all()
    assert (out["v"][0] == bf16_bits(vals[[0, 3]])).all()
    assert abs(out["tau"][0] + ex["cos"][0]) < 1e-14


def test_bf16_widening_is_exact():
    # 0x3F80 = 1, 0xC000 = -2, 0x4049 = 3.140625, 0x3E80 = 0.25 (bf16 = top half of binary32)
    bits = np.array([[0x3F80, 0xC000], [0x4049, 0x3E80], [0x3F80, 0x3F80]], dtype=np.uint16)
    vals = np.array([[1.0, -2.0], [3.140625, 0.25], [1.0, 1.0]])
    N = 2
    kc = np.zeros((1, N, 2), np.uint16); kc[0] = bits[:2]
    out = oracle.evict_units_bf16(kc, kc.copy(), 2, bits[2:][None], bits[2:][None], N)
    # independent cosine-to-anchor of the widened values
    unit = vals / np.linalg.norm(vals, axis=1, keepdims=True)
    mu = unit.mean(0)
    want = unit @ mu / np.linalg.norm(mu)
    np.testing.assert_allclose(-out["e"][0], want, atol=1e-14)


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("m_copies,c", [(1, 0.3), (5, -0.4), (40, 0.9), (7, 0.0), (3, -0.99)])
def test_closed_form_copies_plus_one(m_copies, c):
    # m copies of unit u and one unit w with u.w = c:
    #   cos(u) = (m + c)/D, cos(w) = (m c + 1)/D, D = sqrt(m^2 + 2 m c + 1)
    g = rng(7)
    d = 6
    q, _ = np.linalg.qr(g.standard_normal((d, d)))
    u, t = q[:, 0], q[:, 1]
    w = c * u + math.sqrt(1 - c * c) * t
    scales = g.uniform(0.1, 9.0, size=m_copies + 1)
    K = np.vstack([np.tile(u, (m_copies, 1)), w[None]]) * scales[:, None]
    s = oracle.scores(K)["s"]
    D = math.sqrt(m_copies ** 2 + 2 * m_copies * c + 1)
    np.testing.assert_allclose(s[:-1], (m_copies + c) / D, atol=1e-13)
    assert abs(s[-1] - (m_copies * c + 1) / D) < 1e-13
    # with m > 1 copies and c < 1, w is the most distinctive key: N=1 keeps it
    # (m = 1 is a symmetric pair: both cosines equal (1 + c)/D)
    if m_copies > 1:
        S, _ = oracle.select(oracle.eviction_scores(s), 1)
        assert S.tolist() == [m_copies]


@pytest.mark.parametrize("n,d", [(2, 2), (5, 8), (16, 16), (9, 128)])
def test_closed_form_orthogonal_keys(n, d):
    g = rng(n * 100 + d)
    q, _ = np.linalg.qr(g.standard_normal((d, d)))
    K = q[:, :n].T * g.uniform(0.2, 30.0, size=(n, 1))
    out = oracle.scores(K)
    np.testing.assert_allclose(out["s"], 1 / math.sqrt(n), atol=1e-13)
    assert abs(out["m"] - 1 / math.sqrt(n)) < 1e-13
    np.testing.assert_allclose(out["r"], np.linalg.norm(K, axis=1), rtol=1e-15)


def test_closed_form_identical_directions():
    g = rng(3)
    u = g.standard_normal(128)
    K = np.outer(g.uniform(0.01, 100, size=33), u)
    out = oracle.scores(K)
    np.testing.assert_allclose(out["s"], 1.0, atol=1e-14)
    assert abs(out["m"] - 1.0) < 1e-14


def test_zero_key_scores_zero_and_adds_nothing_to_anchor():
    g = rng(11)
    K = g.standard_normal((9, 16))
    base = oracle.scores(K)
    K0 = np.vstack([K[:4], np.zeros((1, 16)), K[4:]])
    out = oracle.scores(K0)
    assert out["s"][4] == 0.0 and out["r"][4] == 0.0
    # anchor = (sum of the other unit keys)/10 -> same direction, scores of the others unchanged
    np.testing.assert_allclose(out["mu"] * 10, base["mu"] * 9, atol=1e-14)
    np.testing.assert_allclose(np.delete(out["s"], 4), base["s"], atol=1e-14)
    e = oracle.eviction_scores(out["s"])
    assert e[4] == 0.0 and not np.signbit(e[4])       # -0 is canonicalised to +0


def test_eps_clamps_the_product_of_norms():
    # two keys along e1: a unit one and a tiny one (norm 1e-9 < eps = 1e-8).
    # guarded normalisation: k^_1 = 1e-9/max(1e-9, 1e-8) e1 = 0.1 e1, so mu = 0.55 e1, ||mu|| = .55
    # tiny key: mu.k = .55e-9, ||mu||*||k|| = .55e-9 < eps  ->  s = .55e-9/1e-8 = 0.055
    K = np.array([[1.0, 0.0], [1e-9, 0.0]])
    out = oracle.scores(K, eps=1e-8)
    s = out["s"]
    assert abs(out["m"] - 0.55) < 1e-15
    assert abs(s[0] - 1.0) < 1e-15
    assert abs(s[1] - 0.055) < 1e-12
    s = oracle.scores(K, eps=1e-12)["s"]
    assert abs(s[1] - 1.0) < 1e-12


# ---------------------------------------------------------------- identity with the pairwise form
@pytest.mark.parametrize("n,d,seed", [(7, 3, 0), (64, 16, 1), (300, 128, 2)])
def test_pairwise_rowsum_identity(n, d, seed):
    # Eq. (keydiff): rowsum_i(CosSim(K)) = n * ||mu|| * s_i  (App. C derivation), evaluated
    # here with numpy from the definition of the n x n cosine matrix.
    g = rng(seed)
    K = g.standard_normal((n, d)) + 2.0 * g.standard_normal((1, d))
    unit = K / np.sqrt((K * K).sum(1, keepdims=True))
    rowsum = (unit @ unit.T).sum(1)
    out = oracle.scores(K)
    np.testing.assert_allclose(n * out["m"] * out["s"], rowsum, atol=1e-10)
    # the oracle's own literal O(n^2) routine agrees with numpy's
    np.testing.assert_allclose(oracle.pairwise_rowsum(K), rowsum, atol=1e-10)
    # and both rank the tokens identically: same kept sets for several budgets
    e = oracle.eviction_scores(out["s"])
    for N in (1, n // 3, n // 2, n - 1):
        S, _ = oracle.select(e, N)
        S_pair = np.sort(np.argsort(rowsum, kind="stable")[:N])
        assert S.tolist() == S_pair.tolist()


# ---------------------------------------------------------------- brute force on the relaxed objective
@pytest.mark.parametrize("n,d,seed", [(5, 2, 0), (8, 3, 1), (10, 4, 2), (12, 5, 3)])
def test_selection_minimises_relaxed_objective(n, d, seed):
    # Eq. (relaxed_min_cossim_opt): min over |S| = N of sum_{i in S} k^_i . mu(K^), by
    # enumeration of all C(n, N) subsets.
    g = rng(seed)
    K = g.standard_normal((n, d)) + g.standard_normal((1, d))
    unit = K / np.linalg.norm(K, axis=1, keepdims=True)
    obj = unit @ unit.mean(0)
    e = oracle.eviction_scores(oracle.scores(K)["s"])
    for N in range(1, n):
        S, _ = oracle.select(e, N)
        best = min(sum(obj[list(c)]) for c in itertools.combinations(range(n), N))
        assert abs(obj[S].sum() - best) < 1e-12
        assert len(S) == N


# ---------------------------------------------------------------- invariances
def test_scale_invariance():
    g = rng(5)
    K = g.standard_normal((50, 32)) + 1.5
    base = oracle.scores(K)["s"]
    j = g.integers(-8, 9, size=50)
    scaled = oracle.scores(K * (2.0 ** j)[:, None])["s"]
    np.testing.assert_allclose(scaled, base, atol=1e-15)
    e1, e2 = oracle.eviction_scores(base), oracle.eviction_scores(scaled)
    for N in (10, 25, 49):
        assert oracle.select(e1, N)[0].tolist() == oracle.select(e2, N)[0].tolist()


def test_permuting_tokens_permutes_scores():
    g = rng(6)
    K = g.standard_normal((40, 16)) + 1.0
    p = g.permutation(40)
    np.testing.assert_allclose(oracle.scores(K[p])["s"], oracle.scores(K)["s"][p], atol=1e-14)


# ---------------------------------------------------------------- selection rule
@pytest.mark.parametrize("seed", range(5))
def test_select_properties(seed):
    g = rng(seed)
    n = 200
    e = np.round(g.standard_normal(n), 1)            # many exact ties
    for N in (1, 17, 100, 199, 200, 250):
        S, tau = oracle.select(e, N)
        assert len(S) == min(N, n)
        assert (np.diff(S) > 0).all()                 # ascending = original token order
        kept = np.zeros(n, bool); kept[S] = True
        if kept.all():
            continue
        assert e[kept].min() >= e[~kept].max()        # every kept score >= every evicted score
        assert tau == e[kept].min()
        # among tokens tied at the threshold, the kept ones are the oldest
        tied = np.flatnonzero(e == tau)
        k_t, ev_t = tied[kept[tied]], tied[~kept[tied]]
        if len(k_t) and len(ev_t):
            assert k_t.max() < ev_t.min()


def test_select_matches_exhaustive_definition_on_tiny_inputs():
    # all 3^5 score vectors over {-1,0,1}: compare with a literal ranking by (e desc, i asc)
    for e in itertools.product([-1.0, 0.0, 1.0], repeat=5):
        e = np.array(e)
        ranked = sorted(range(5), key=lambda i: (-e[i], i))
        for N in range(1, 5):
            assert oracle.select(e, N)[0].tolist() == sorted(ranked[:N])


# ---------------------------------------------------------------- the step (append / evict / gather)
def _units(U, length, B, N, d, seed):
    g = rng(seed)
    kc = np.zeros((U, N, d), np.float32); vc = np.zeros((U, N, d), np.float32)
    kc[:, :length] = g.standard_normal((U, length, d)) + 1.0
    vc[:, :length] = g.standard_normal((U, length, d))
    nk = (g.standard_normal((U, B, d)) + 1.0).astype(np.float32)
    nv = g.standard_normal((U, B, d)).astype(np.float32)
    return bf16_bits(kc), bf16_bits(vc), bf16_bits(nk), bf16_bits(nv)


def test_append_only_when_budget_not_exceeded():
    kc, vc, nk, nv = _units(3, 10, 6, 16, 8, 0)      # 10 + 6 = 16 <= N
    out = oracle.evict_units_bf16(kc, vc, 10, nk, nv, 16)
    assert out["len"] == 16 and out["e"] is None
    assert (out["k"][:, :10] == kc[:, :10]).all() and (out["k"][:, 10:16] == nk).all()
    assert (out["v"][:, :10] == vc[:, :10]).all() and (out["v"][:, 10:16] == nv).all()


@pytest.mark.parametrize("length,B,N", [(16, 4, 16), (13, 8, 16), (16, 1, 16), (0, 40, 16)])
def test_evicting_step_invariants(length, B, N):
    U, d = 4, 8
    kc, vc, nk, nv = _units(U, length, B, N, d, 1)
    out = oracle.evict_units_bf16(kc, vc, length, nk, nv, N)
    n = length + B
    assert out["len"] == N == out["S"].shape[1]
    for u in range(U):
        allk = np.concatenate([kc[u, :length], nk[u]]); allv = np.concatenate([vc[u, :length], nv[u]])
        S = out["S"][u]
        assert (np.diff(S) > 0).all() and S.min() >= 0 and S.max() < n
        assert (out["k"][u] == allk[S]).all() and (out["v"][u] == allv[S]).all()   # bit-exact, paired
        kept = np.zeros(n, bool); kept[S] = True
        assert out["e"][u][kept].min() >= out["e"][u][~kept].max()
        assert out["tau"][u] == out["e"][u][kept].min()


def test_single_block_equals_whole_prompt():
    # B = T: one step over the whole prompt is the function applied to all keys at once
    U, T, N, d = 2, 40, 16, 8
    kc, vc, nk, nv = _units(U, 0, T, N, d, 2)
    out = oracle.evict_units_bf16(kc, vc, 0, nk, nv, N)
    for u in range(U):
        K = torch.from_numpy(nk[u].view(np.int16)).view(torch.bfloat16).double().numpy()
        e = oracle.eviction_scores(oracle.scores(K)["s"])
        assert out["S"][u].tolist() == oracle.select(e, N)[0].tolist()


def test_threads_do_not_change_results():
    kc, vc, nk, nv = _units(9, 32, 8, 32, 16, 3)
    a = oracle.evict_units_bf16(kc, vc, 32, nk, nv, 32, n_threads=1)
    b = oracle.evict_units_bf16(kc, vc, 32, nk, nv, 32, n_threads=4)
    assert a["threads"] == 1 and b["threads"] == 4
    for key in ("k", "v", "e", "S", "tau", "m"):
        assert (a[key] == b[key]).all()


def test_block_streaming_keeps_budget_and_order():
    # Eq. (block_processing): C_0 empty, append block, apply pi_N, carry on.  Values carry the
    # token position so order and K/V pairing can be read back.
    U, N, B, d, T = 2, 24, 8, 8, 96
    g = rng(4)
    keys = (g.standard_normal((U, T, d)) + 1.0).astype(np.float32)
    vals = np.broadcast_to(np.arange(T, dtype=np.float32)[None, :, None], (U, T, d)).copy()
    kc = np.zeros((U, N, d), np.uint16); vc = np.zeros((U, N, d), np.uint16)
    length = 0
    for t0 in range(0, T, B):
        out = oracle.evict_units_bf16(kc, vc, length, bf16_bits(keys[:, t0:t0 + B]),
                                      bf16_bits(vals[:, t0:t0 + B]), N)
        kc, vc, length = out["k"], out["v"], out["len"]
        assert length == min(N, t0 + B)
        pos = torch.from_numpy(vc[:, :length, 0].view(np.int16).copy()).view(torch.bfloat16).float().numpy()
        assert (np.diff(pos, axis=1) > 0).all()                     # original token order kept
        for u in range(U):                                          # K rows still paired with V rows
            assert (kc[u, :length] == bf16_bits(keys[u, pos[u].astype(int)])).all()
