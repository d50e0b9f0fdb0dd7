"""Acceptance rules for comparing a CUDA eviction step with the CPU oracle.
TEST INFRASTRUCTURE, NOT PRODUCT CODE (imported by tests, the smoke check and the benchmark's
verification leg only).

Rules (per unit, one evicting step, both sides fed the same bf16 bits):
  scores     |e_gpu - e_ref| <= 1e-5 * max(|e_ref|, kappa_i), kappa_i = sum_c|mu_c k_ic| / (||mu|| ||k_i||)
             (the magnitude of the terms of the dot product: a cosine near 0 is a cancelling sum,
             so a purely relative bound on it is unattainable in any finite precision), and the
             plain relative error <= 1e-5 wherever |e_ref| >= 1e-2.  Required when ||mu|| >= 1e-3.
  selection  exactly N kept; the kept set is the top-N of the GPU's OWN fp32 scores under
             (e desc, index asc) -- bit exact; and it agrees with the oracle's set on every token
             whose oracle score is more than 1e-5 away from the oracle's threshold tau.
  gather     kept rows of K and V are bit-exact copies of the source rows, in token order.
"""
from __future__ import annotations

import numpy as np

from . import oracle

SCORE_RTOL = 1e-5
TAU_BAND = 1e-5
PLAIN_REL_FLOOR = 1e-2
MIN_ANCHOR_NORM = 1e-3


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def check_step(k_cache, v_cache, length, new_k, new_v, N, gpu_k, gpu_v, gpu_scores, gpu_kept,
               eps=oracle.DEFAULT_EPS, units=None, n_threads=1, anchor_mode=0, recent_window=0):
    """All array arguments are host numpy arrays: uint16 bit patterns [U, rows, d] for K/V,
    float32 [U, >=n] for gpu_scores, int32 [U, N] for gpu_kept.  ``units`` restricts the check to
    a subset of unit indices.  anchor_mode / recent_window select the method's variants (raw-mean anchor;
    the last recent_window tokens always kept).  Returns a report dict; raises AssertionError on a violation."""
    U = k_cache.shape[0]
    sel = np.arange(U) if units is None else np.asarray(units)
    B = new_k.shape[1]
    n = length + B
    assert n > N, "check_step is for evicting steps"
    ref = oracle.evict_units_bf16(k_cache[sel], v_cache[sel], length, new_k[sel], new_v[sel], N, eps, n_threads,
                                  anchor_mode=anchor_mode, recent_window=recent_window)
    w = recent_window
    rep = {"units": len(sel), "n": n, "max_score_err_over_tol": 0.0, "max_plain_rel": 0.0,
           "set_mismatch_in_band": 0, "min_anchor_norm": float(ref["m"].min()),
           "max_plain_rel_all_tokens": 0.0, "frac_tokens_below_floor": 0.0}
    for j, u in enumerate(sel):
        allk = np.concatenate([k_cache[u, :length], new_k[u]])
        allv = np.concatenate([v_cache[u, :length], new_v[u]])
        e_ref = ref["e"][j]
        e_gpu = gpu_scores[u, :n].astype(np.float64)
        assert np.isfinite(e_gpu).all(), f"unit {u}: non-finite GPU score"
        # ---- scores
        if ref["m"][j] >= MIN_ANCHOR_NORM:
            K = _bf16_to_f64(allk)
            r = np.sqrt((K * K).sum(1))
            unit = K if anchor_mode == 1 else K / np.maximum(r, eps)[:, None]
            mu = unit.sum(0) / n
            kappa = (np.abs(K) @ np.abs(mu)) / np.maximum(np.sqrt((mu * mu).sum()) * r, eps)
            tol = SCORE_RTOL * np.maximum(np.abs(e_ref), kappa)
            err = np.abs(e_gpu - e_ref)
            worst = float((err / np.maximum(tol, 1e-300)).max())
            rep["max_score_err_over_tol"] = max(rep["max_score_err_over_tol"], worst)
            assert worst <= 1.0, f"unit {u}: score error {worst:.3f}x the tolerance"
            big = np.abs(e_ref) >= PLAIN_REL_FLOOR
            if big.any():
                rel = float((err[big] / np.abs(e_ref[big])).max())
                rep["max_plain_rel"] = max(rep["max_plain_rel"], rel)
                assert rel <= SCORE_RTOL, f"unit {u}: plain relative score error {rel:.3e}"
            # reported, not asserted: how far the plain relative rule is missed on the scores below the floor
            nz = e_ref != 0
            if nz.any():
                rep["max_plain_rel_all_tokens"] = max(rep["max_plain_rel_all_tokens"], float((err[nz] / np.abs(e_ref[nz])).max()))
            rep["frac_tokens_below_floor"] += float((~big).mean()) / len(sel)
        # ---- selection: exact w.r.t. the GPU's own scores
        S_gpu = gpu_kept[u].astype(np.int64)
        assert len(S_gpu) == N and (np.diff(S_gpu) > 0).all() and S_gpu[0] >= 0 and S_gpu[-1] < n, \
            f"unit {u}: kept list is not N ascending in-range indices"
        e32 = gpu_scores[u, :n]
        head = n - w                                                     # tokens the score rule decides on
        order = np.lexsort((np.arange(head), -e32[:head].astype(np.float64)))     # e desc, index asc
        want = np.sort(np.concatenate([order[:N - w], np.arange(head, n)]))
        assert (S_gpu == want).all(), f"unit {u}: kept set is not the top-N of the GPU's own scores"
        # ---- selection: agreement with the oracle outside the threshold band
        S_ref = ref["S"][j]
        if not (S_gpu == S_ref).all():
            diff = np.setxor1d(S_gpu, S_ref)
            dist = np.abs(e_ref[diff] - ref["tau"][j])
            assert (dist <= TAU_BAND).all(), \
                f"unit {u}: kept sets differ on tokens {diff[dist > TAU_BAND][:8]} outside the tau band"
            rep["set_mismatch_in_band"] += len(diff)
        # ---- gather: bit-exact rows in token order
        assert (gpu_k[u, :N] == allk[S_gpu]).all(), f"unit {u}: K rows are not bit-exact copies"
        assert (gpu_v[u, :N] == allv[S_gpu]).all(), f"unit {u}: V rows are not bit-exact copies"
        if (S_gpu == S_ref).all():
            assert (gpu_k[u, :N] == ref["k"][j]).all() and (gpu_v[u, :N] == ref["v"][j]).all()
    return rep


def check_step_slots(k_cache, v_cache, pos, next_pos, length, new_k, new_v, N, gpu_k, gpu_v, gpu_scores, gpu_src,
                     gpu_pos, eps=oracle.DEFAULT_EPS, units=None, n_threads=1, anchor_mode=0, recent_window=0):
    """The same acceptance rules for a step with unordered slot reuse.  pos: int [U, N] token positions of
    the slots before the step; gpu_src: int32 [U, N], the candidate number each slot holds after it (the
    library's kept_idx in this mode); gpu_pos: int32 [U, N] positions after it.
      scores     as in check_step;
      selection  the kept candidates are the top-N of the GPU's own fp32 scores under (e desc, candidate
                 number asc), tokens at the last recent_window positions always kept; agreement with the
                 oracle outside the tau band;
      placement  kept cache rows untouched; the kept block rows, in block order, in the freed slots in
                 ascending order; rows bit-exact; positions exact."""
    U = k_cache.shape[0]
    sel = np.arange(U) if units is None else np.asarray(units)
    B = new_k.shape[1]
    n = length + B
    assert n > N, "check_step_slots is for evicting steps"
    ref = oracle.evict_units_bf16_slots(k_cache[sel], v_cache[sel], pos[sel], length, next_pos, new_k[sel], new_v[sel], N,
                                        eps, n_threads, anchor_mode=anchor_mode, recent_window=recent_window)
    rep = {"units": len(sel), "n": n, "max_score_err_over_tol": 0.0, "max_plain_rel": 0.0,
           "set_mismatch_in_band": 0, "min_anchor_norm": float(ref["m"].min()),
           "max_plain_rel_all_tokens": 0.0, "frac_tokens_below_floor": 0.0}
    for j, u in enumerate(sel):
        allk = np.concatenate([k_cache[u, :length], new_k[u]])
        allv = np.concatenate([v_cache[u, :length], new_v[u]])
        cand_pos = np.concatenate([pos[u, :length].astype(np.int64), next_pos + np.arange(B)])
        e_ref = ref["e"][j]
        e_gpu = gpu_scores[u, :n].astype(np.float64)
        assert np.isfinite(e_gpu).all(), f"unit {u}: non-finite GPU score"
        if ref["m"][j] >= MIN_ANCHOR_NORM:
            K = _bf16_to_f64(allk)
            r = np.sqrt((K * K).sum(1))
            unit = K if anchor_mode == 1 else K / np.maximum(r, eps)[:, None]
            mu = unit.sum(0) / n
            kappa = (np.abs(K) @ np.abs(mu)) / np.maximum(np.sqrt((mu * mu).sum()) * r, eps)
            tol = SCORE_RTOL * np.maximum(np.abs(e_ref), kappa)
            err = np.abs(e_gpu - e_ref)
            worst = float((err / np.maximum(tol, 1e-300)).max())
            rep["max_score_err_over_tol"] = max(rep["max_score_err_over_tol"], worst)
            assert worst <= 1.0, f"unit {u}: score error {worst:.3f}x the tolerance"
            big = np.abs(e_ref) >= PLAIN_REL_FLOOR
            if big.any():
                rel = float((err[big] / np.abs(e_ref[big])).max())
                rep["max_plain_rel"] = max(rep["max_plain_rel"], rel)
                assert rel <= SCORE_RTOL, f"unit {u}: plain relative score error {rel:.3e}"
            nz = e_ref != 0
            if nz.any():
                rep["max_plain_rel_all_tokens"] = max(rep["max_plain_rel_all_tokens"], float((err[nz] / np.abs(e_ref[nz])).max()))
            rep["frac_tokens_below_floor"] += float((~big).mean()) / len(sel)
        # ---- selection w.r.t. the GPU's own scores
        src = gpu_src[u].astype(np.int64)
        assert len(set(src.tolist())) == N and src.min() >= 0 and src.max() < n, f"unit {u}: slots do not hold N distinct candidates"
        recent = cand_pos >= next_pos + B - recent_window
        rest = np.nonzero(~recent)[0]
        e32 = gpu_scores[u, :n]
        order = rest[np.lexsort((rest, -e32[rest].astype(np.float64)))]
        want = np.sort(np.concatenate([order[:max(N - int(recent.sum()), 0)], np.nonzero(recent)[0]]))
        S_gpu = np.sort(src)
        assert (S_gpu == want).all(), f"unit {u}: kept candidates are not the top-N of the GPU's own scores"
        # ---- agreement with the oracle outside the threshold band
        S_ref = np.sort(ref["src"][j])
        if not (S_gpu == S_ref).all():
            diff = np.setxor1d(S_gpu, S_ref)
            dist = np.abs(e_ref[diff] - ref["tau"][j])
            assert (dist <= TAU_BAND).all(), f"unit {u}: kept sets differ on candidates {diff[dist > TAU_BAND][:8]} outside the tau band"
            rep["set_mismatch_in_band"] += len(diff)
        # ---- placement, given the kept set
        kept = np.zeros(n, dtype=bool); kept[S_gpu] = True
        free = np.concatenate([np.nonzero(~kept[:length])[0], np.arange(length, N)])
        blocks = length + np.nonzero(kept[length:])[0]
        assert len(free) == len(blocks)
        exp_src = np.arange(N); exp_src[free] = blocks
        assert (src == exp_src).all(), f"unit {u}: block rows are not in the freed slots in order"
        assert (gpu_pos[u].astype(np.int64) == cand_pos[exp_src]).all(), f"unit {u}: slot positions are wrong"
        assert (gpu_k[u, :N] == allk[exp_src]).all(), f"unit {u}: K rows are not bit-exact copies"
        assert (gpu_v[u, :N] == allv[exp_src]).all(), f"unit {u}: V rows are not bit-exact copies"
        if (S_gpu == S_ref).all():
            assert (gpu_k[u, :N] == ref["k"][j]).all() and (gpu_v[u, :N] == ref["v"][j]).all()
            assert (gpu_pos[u] == ref["pos"][j]).all()
    return rep
