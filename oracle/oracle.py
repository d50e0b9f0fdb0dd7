"""ctypes loader for the KeyDiff CPU oracle.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this module.  It compiles ``keydiff_oracle.cpp`` with g++ into
``libkeydiff_oracle.so`` next to the source and exposes numpy-typed wrappers; no
arithmetic of the method lives here (argument marshalling only).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "keydiff_oracle.cpp"
_LIB = _HERE / "libkeydiff_oracle.so"
_lib = None

DEFAULT_EPS = 1e-8


def build(force: bool = False) -> Path:
    """Compile the oracle (g++ -O2, no fast-math) if the .so is missing or stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread",
               "-fno-fast-math", "-ffp-contract=off", str(_SRC), "-o", str(tmp)]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        c_dp = ctypes.POINTER(ctypes.c_double)
        c_ip = ctypes.POINTER(ctypes.c_int64)
        c_hp = ctypes.POINTER(ctypes.c_uint16)
        i64, f64 = ctypes.c_int64, ctypes.c_double
        lib.kd_oracle_scores.argtypes = [c_dp, i64, i64, f64, c_dp, c_dp, c_dp, c_dp]
        lib.kd_oracle_scores.restype = None
        lib.kd_oracle_eviction_scores.argtypes = [c_dp, i64, c_dp]
        lib.kd_oracle_eviction_scores.restype = None
        lib.kd_oracle_select.argtypes = [c_dp, i64, i64, c_ip, c_dp]
        lib.kd_oracle_select.restype = i64
        lib.kd_oracle_pairwise_rowsum.argtypes = [c_dp, i64, i64, c_dp]
        lib.kd_oracle_pairwise_rowsum.restype = None
        lib.kd_oracle_evict_head_bf16.argtypes = [c_hp, c_hp, i64, c_hp, c_hp, i64, i64, i64, f64,
                                                  c_hp, c_hp, c_ip, c_dp, c_ip, c_dp, c_dp]
        lib.kd_oracle_evict_head_bf16.restype = None
        lib.kd_oracle_evict_units_bf16.argtypes = [c_hp, c_hp, i64, c_hp, c_hp, i64, i64, i64, f64, i64,
                                                   c_hp, c_hp, c_dp, c_ip, c_dp, c_dp, ctypes.c_int32]
        lib.kd_oracle_evict_units_bf16.restype = ctypes.c_int32
        lib.kd_oracle_scores_ex.argtypes = [c_dp, i64, i64, f64, ctypes.c_int32, c_dp, c_dp, c_dp, c_dp]
        lib.kd_oracle_scores_ex.restype = None
        lib.kd_oracle_select_window.argtypes = [c_dp, i64, i64, i64, c_ip, c_dp]
        lib.kd_oracle_select_window.restype = i64
        lib.kd_oracle_evict_units_bf16_ex.argtypes = [c_hp, c_hp, i64, c_hp, c_hp, i64, i64, i64, f64, i64,
                                                      ctypes.c_int32, i64, c_hp, c_hp, c_dp, c_ip, c_dp, c_dp]
        lib.kd_oracle_evict_units_bf16_ex.restype = None
        lib.kd_oracle_evict_units_bf16_slots.argtypes = [c_hp, c_hp, c_ip, i64, i64, c_hp, c_hp, i64, i64, i64, f64, i64,
                                                         ctypes.c_int32, i64, c_hp, c_hp, c_ip, c_ip, c_dp, c_dp, c_dp]
        lib.kd_oracle_evict_units_bf16_slots.restype = None
        _lib = lib
    return _lib


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _hp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def scores(K, eps: float = DEFAULT_EPS, anchor_mode: int = 0):
    """K: (n, d) float64.  Returns dict r (n,), mu (d,), m (float), s (n,) cosines.
    anchor_mode 0: anchor = mean of normalised keys; 1: mean of the raw keys."""
    K = np.ascontiguousarray(K, dtype=np.float64)
    n, d = K.shape
    r, mu, s = np.empty(n), np.empty(d), np.empty(n)
    m = np.empty(1)
    _load().kd_oracle_scores_ex(_dp(K), n, d, eps, anchor_mode, _dp(r), _dp(mu), _dp(m), _dp(s))
    return {"r": r, "mu": mu, "m": float(m[0]), "s": s}


def eviction_scores(s):
    s = np.ascontiguousarray(s, dtype=np.float64)
    e = np.empty_like(s)
    _load().kd_oracle_eviction_scores(_dp(s), s.size, _dp(e))
    return e


def select(e, N: int, recent_window: int = 0):
    """Kept token indices (ascending) and the threshold tau (score of the last token the score rule
    keeps).  recent_window w: the last w tokens are always kept, the rest compete for N - w places."""
    e = np.ascontiguousarray(e, dtype=np.float64)
    keep = min(N, e.size)
    S = np.empty(keep, dtype=np.int64)
    tau = np.empty(1)
    got = _load().kd_oracle_select_window(_dp(e), e.size, N, recent_window, _ip(S), _dp(tau))
    assert got == keep
    return S, float(tau[0])


def pairwise_rowsum(K):
    K = np.ascontiguousarray(K, dtype=np.float64)
    n, d = K.shape
    out = np.empty(n)
    _load().kd_oracle_pairwise_rowsum(_dp(K), n, d, _dp(out))
    return out


def evict_units_bf16(k_cache, v_cache, length: int, new_k, new_v, N: int,
                     eps: float = DEFAULT_EPS, n_threads: int = 1, anchor_mode: int = 0, recent_window: int = 0):
    """U independent units on bf16 bit patterns (uint16 arrays).

    k_cache, v_cache: (U, N, d) uint16 with rows [0, length) valid; new_k, new_v:
    (U, B, d) uint16.  Returns dict: k, v (U, N, d) uint16 with rows [0, len) valid,
    len (int), e (U, n) float64 or None when nothing was evicted, S (U, len) int64,
    tau (U,), m (U,), threads (int actually used).
    """
    k_cache = np.ascontiguousarray(k_cache, dtype=np.uint16)
    v_cache = np.ascontiguousarray(v_cache, dtype=np.uint16)
    new_k = np.ascontiguousarray(new_k, dtype=np.uint16)
    new_v = np.ascontiguousarray(new_v, dtype=np.uint16)
    U, cap, d = k_cache.shape
    assert cap == N and v_cache.shape == k_cache.shape
    B = new_k.shape[1]
    assert new_k.shape == (U, B, d) and new_v.shape == (U, B, d)
    assert 0 <= length <= N
    n = length + B
    keep = min(N, n)
    k_out = np.zeros((U, N, d), dtype=np.uint16)
    v_out = np.zeros((U, N, d), dtype=np.uint16)
    e = np.zeros((U, n), dtype=np.float64)
    S_full = np.zeros((U, N), dtype=np.int64)
    tau, m = np.zeros(U), np.zeros(U)
    if anchor_mode == 0 and recent_window == 0:
        used = _load().kd_oracle_evict_units_bf16(
            _hp(k_cache), _hp(v_cache), length, _hp(new_k), _hp(new_v), B, N, d, eps, U,
            _hp(k_out), _hp(v_out), _dp(e), _ip(S_full), _dp(tau), _dp(m), n_threads)
    else:
        assert 0 <= recent_window <= N
        from concurrent.futures import ThreadPoolExecutor
        used = max(1, min(n_threads, U))
        lib = _load()

        def run(t):   # units t, t+used, ...: one C call per unit (ctypes drops the GIL)
            for u in range(t, U, used):
                lib.kd_oracle_evict_units_bf16_ex(
                    _hp(k_cache[u]), _hp(v_cache[u]), length, _hp(new_k[u]), _hp(new_v[u]), B, N, d, eps, 1,
                    anchor_mode, recent_window, _hp(k_out[u]), _hp(v_out[u]), _dp(e[u]), _ip(S_full[u]),
                    _dp(tau[u:u + 1]), _dp(m[u:u + 1]))
        with ThreadPoolExecutor(used) as pool:
            list(pool.map(run, range(used)))
    return {"k": k_out, "v": v_out, "len": keep, "e": e if n > N else None,
            "S": S_full[:, :keep].copy(), "tau": tau, "m": m, "threads": int(used)}


def evict_units_bf16_slots(k_cache, v_cache, pos, length: int, next_pos: int, new_k, new_v, N: int,
                           eps: float = DEFAULT_EPS, n_threads: int = 1, anchor_mode: int = 0, recent_window: int = 0):
    """U units with unordered slot reuse: kept cache rows stay in their slots, kept block rows fill
    the freed slots.  pos: (U, N) int64, the token position held by each of the `length` valid slots;
    the block rows are tokens next_pos .. next_pos + B - 1.

    Returns dict: k, v (U, N, d) uint16, pos (U, N) int64, src (U, N) int64 (candidate number now in
    each slot: the slot itself for a cache row, length + j for block row j), len, e (U, n) or None,
    tau, m, threads.
    """
    k_cache = np.ascontiguousarray(k_cache, dtype=np.uint16)
    v_cache = np.ascontiguousarray(v_cache, dtype=np.uint16)
    new_k = np.ascontiguousarray(new_k, dtype=np.uint16)
    new_v = np.ascontiguousarray(new_v, dtype=np.uint16)
    pos = np.ascontiguousarray(pos, dtype=np.int64)
    U, cap, d = k_cache.shape
    B = new_k.shape[1]
    assert cap == N and v_cache.shape == k_cache.shape and pos.shape == (U, N)
    assert new_k.shape == (U, B, d) and new_v.shape == (U, B, d)
    assert 0 <= length <= N and 0 <= recent_window <= N
    n = length + B
    k_out = np.zeros((U, N, d), dtype=np.uint16)
    v_out = np.zeros((U, N, d), dtype=np.uint16)
    pos_out = np.zeros((U, N), dtype=np.int64)
    src = np.zeros((U, N), dtype=np.int64)
    e = np.zeros((U, n), dtype=np.float64)
    tau, m = np.zeros(U), np.zeros(U)
    from concurrent.futures import ThreadPoolExecutor
    used = max(1, min(n_threads, U))
    lib = _load()

    def run(t):
        for u in range(t, U, used):
            lib.kd_oracle_evict_units_bf16_slots(
                _hp(k_cache[u]), _hp(v_cache[u]), _ip(pos[u]), length, next_pos, _hp(new_k[u]), _hp(new_v[u]),
                B, N, d, eps, 1, anchor_mode, recent_window, _hp(k_out[u]), _hp(v_out[u]), _ip(pos_out[u]),
                _ip(src[u]), _dp(e[u]), _dp(tau[u:u + 1]), _dp(m[u:u + 1]))
    with ThreadPoolExecutor(used) as pool:
        list(pool.map(run, range(used)))
    return {"k": k_out, "v": v_out, "pos": pos_out, "src": src, "len": min(N, n), "e": e if n > N else None,
            "tau": tau, "m": m, "threads": int(used)}
