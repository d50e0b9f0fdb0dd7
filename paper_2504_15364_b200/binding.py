"""Thin ctypes binding over ``libkeydiff.so`` (the C ABI of include/keydiff.h).

Argument marshalling only: every step of the eviction path runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  There is no CPU fallback: if the
shared library is missing or no sm_100 device is present, loading / creating raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libkeydiff.so"

KEYDIFF_OK = 0
KEYDIFF_ERR_INVALID_ARG, KEYDIFF_ERR_UNSUPPORTED, KEYDIFF_ERR_ALLOC = -1, -2, -3
KEYDIFF_ERR_CUDA, KEYDIFF_ERR_STATE, KEYDIFF_ERR_TIMEOUT = -4, -5, -6
KEYDIFF_ERR_TOO_LARGE = -7
KEYDIFF_ERR_INTERNAL = -8
KEYDIFF_BF16 = 0
KEYDIFF_PATH_AUTO, KEYDIFF_PATH_STAGED, KEYDIFF_PATH_FUSED = 0, 1, 2
KEYDIFF_ANCHOR_NORMALISED, KEYDIFF_ANCHOR_RAW_MEAN = 0, 1
KEYDIFF_COMPACT_ORDERED, KEYDIFF_COMPACT_SLOT_REUSE = 0, 1

# every symbol include/keydiff.h declares
EXPORTS = ["keydiff_create", "keydiff_evict", "keydiff_evict_host", "keydiff_destroy", "keydiff_reset",
           "keydiff_get_len", "keydiff_set_len", "keydiff_get_scratch", "keydiff_get_moved_rows",
           "keydiff_get_launch_info", "keydiff_evict_static", "keydiff_set_incremental", "keydiff_get_positions",
           "keydiff_set_positions", "keydiff_selftest_bounded_wait", "keydiff_debug_fail_alloc",
           "keydiff_strerror", "keydiff_last_cuda_error"]


class keydiff_config(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("budget", ctypes.c_int32), ("max_block", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("path", ctypes.c_int32), ("eps", ctypes.c_float),
                ("device", ctypes.c_int32), ("anchor_mode", ctypes.c_int32), ("recent_window", ctypes.c_int32),
                ("compaction", ctypes.c_int32)]


class KeyDiffError(RuntimeError):
    def __init__(self, code: int, text: str, cuda_error: int = 0):
        super().__init__(f"keydiff: {text} (status {code}" + (f", cudaError {cuda_error})" if cuda_error else ")"))
        self.code = code
        self.cuda_error = cuda_error


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen the in-tree library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise KeyDiffError(KEYDIFF_ERR_STATE, f"{LIB_PATH} not built: run `python -m paper_2504_15364_b200.build`")
    lib = ctypes.CDLL(str(LIB_PATH))
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    i32p = ctypes.POINTER(ctypes.c_int32)
    lib.keydiff_create.argtypes = [ctypes.POINTER(keydiff_config), ctypes.POINTER(vp)]
    lib.keydiff_evict.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.keydiff_evict_host.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp]
    lib.keydiff_destroy.argtypes = [vp]
    lib.keydiff_reset.argtypes = [vp]
    lib.keydiff_get_len.argtypes = [vp, i32p]
    lib.keydiff_set_len.argtypes = [vp, i32]
    lib.keydiff_set_incremental.argtypes = [vp, i32]
    lib.keydiff_get_scratch.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.keydiff_get_moved_rows.argtypes = [vp, ctypes.POINTER(vp)]
    lib.keydiff_get_positions.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_longlong)]
    lib.keydiff_set_positions.argtypes = [vp, vp, i32, ctypes.c_longlong, vp]
    lib.keydiff_selftest_bounded_wait.argtypes = [vp, i32, vp]
    lib.keydiff_debug_fail_alloc.argtypes = [i32]
    lib.keydiff_get_launch_info.argtypes = [vp, i32p, i32p, i32p]
    lib.keydiff_evict_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, ctypes.c_float, vp]
    lib.keydiff_strerror.argtypes = [ctypes.c_int]
    lib.keydiff_strerror.restype = ctypes.c_char_p
    lib.keydiff_last_cuda_error.argtypes = []
    for name in EXPORTS:
        if name != "keydiff_strerror":
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(rc: int):
    if rc != KEYDIFF_OK:
        lib = load_library()
        raise KeyDiffError(rc, lib.keydiff_strerror(rc).decode(), lib.keydiff_last_cuda_error())


class _DevArray:
    """Exposes a raw device pointer through __cuda_array_interface__ so torch can view it."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False),
                                         "version": 2, "strides": None}


class KeyDiff:
    """One eviction context: U = n_layers*batch*n_kv_heads independent units, budget N.

    ``evict`` mirrors ``keydiff_evict``; tensors are bf16 CUDA tensors laid out
    [n_layers, batch, n_kv_heads, rows, head_dim] (or the same flattened to [U, rows, head_dim]).
    ``anchor_mode`` / ``recent_window`` choose the method's variants (raw-mean anchor, sliding window);
    ``compaction=KEYDIFF_COMPACT_SLOT_REUSE`` leaves kept cache rows in their slots and writes the kept
    block rows into the freed ones (``positions()`` then tells which token each slot holds).
    """

    def __init__(self, n_layers: int, batch: int, n_kv_heads: int, head_dim: int, budget: int, max_block: int,
                 *, path: int = KEYDIFF_PATH_AUTO, eps: float = 0.0, device: int | None = None,
                 anchor_mode: int = KEYDIFF_ANCHOR_NORMALISED, recent_window: int = 0,
                 compaction: int = KEYDIFF_COMPACT_ORDERED):
        self._lib = load_library()
        self._ctx = ctypes.c_void_p()
        if device is None:
            device = torch.cuda.current_device() if torch.cuda.is_available() else 0
        self.cfg = keydiff_config(n_layers, batch, n_kv_heads, head_dim, budget, max_block, KEYDIFF_BF16, path,
                                  eps, device, anchor_mode, recent_window, compaction)
        _check(self._lib.keydiff_create(ctypes.byref(self.cfg), ctypes.byref(self._ctx)))
        self.units = n_layers * batch * n_kv_heads
        self.budget, self.max_block, self.head_dim, self.n_kv_heads = budget, max_block, head_dim, n_kv_heads
        self.device = torch.device("cuda", device)

    # -- the step ---------------------------------------------------------------------------
    def _check_tensor(self, t: torch.Tensor, rows: int, name: str):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
            raise KeyDiffError(KEYDIFF_ERR_INVALID_ARG, f"{name}: need a contiguous bf16 CUDA tensor")
        if t.numel() != self.units * rows * self.head_dim:
            raise KeyDiffError(KEYDIFF_ERR_INVALID_ARG, f"{name}: expected {self.units}x{rows}x{self.head_dim} elements")

    def evict(self, k_cache, v_cache, new_k, new_v, stream: torch.cuda.Stream | None = None) -> int:
        """Append the block and evict back to the budget, in place.  Returns the new length."""
        B = new_k.numel() // (self.units * self.head_dim)
        self._check_tensor(k_cache, self.budget, "k_cache"); self._check_tensor(v_cache, self.budget, "v_cache")
        self._check_tensor(new_k, B, "new_k"); self._check_tensor(new_v, B, "new_v")
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self._lib.keydiff_evict(self._ctx, k_cache.data_ptr(), v_cache.data_ptr(), new_k.data_ptr(),
                                       new_v.data_ptr(), self.budget, B, self.n_kv_heads, self.head_dim, st))
        return self.len

    def evict_host(self, k_cache, v_cache, new_k_host, new_v_host, kept_idx_host=None, status_host=None,
                   stream: torch.cuda.Stream | None = None) -> int:
        """Same step with the block in (pinned) host memory; optionally reads the kept-index list
        (int32 [U, N]) and the status word back into host tensors."""
        B = new_k_host.numel() // (self.units * self.head_dim)
        self._check_tensor(k_cache, self.budget, "k_cache"); self._check_tensor(v_cache, self.budget, "v_cache")
        for t in (new_k_host, new_v_host):
            if t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
                raise KeyDiffError(KEYDIFF_ERR_INVALID_ARG, "host block: need a contiguous bf16 CPU tensor")
        if kept_idx_host is not None:
            assert kept_idx_host.dtype == torch.int32 and kept_idx_host.numel() == self.units * self.budget
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self._lib.keydiff_evict_host(
            self._ctx, k_cache.data_ptr(), v_cache.data_ptr(), new_k_host.data_ptr(), new_v_host.data_ptr(),
            self.budget, B, self.n_kv_heads, self.head_dim,
            kept_idx_host.data_ptr() if kept_idx_host is not None else None,
            status_host.data_ptr() if status_host is not None else None, st))
        return self.len

    # -- bookkeeping ------------------------------------------------------------------------
    @property
    def len(self) -> int:
        out = ctypes.c_int32()
        _check(self._lib.keydiff_get_len(self._ctx, ctypes.byref(out)))
        return out.value

    def set_len(self, n: int):
        _check(self._lib.keydiff_set_len(self._ctx, n))

    def reset(self):
        _check(self._lib.keydiff_reset(self._ctx))

    def set_incremental(self, on: bool):
        """``keydiff_set_incremental``: keep the anchor's running sum across steps (default) or rebuild it every step."""
        _check(self._lib.keydiff_set_incremental(self._ctx, 1 if on else 0))

    def scratch(self):
        """Views (no copy) of the ctx-owned scratch: scores [U, N+max_block] fp32, kept_idx [U, N]
        int32, first_evicted [U] int32, status [1] int32."""
        p = [ctypes.c_void_p() for _ in range(4)]
        _check(self._lib.keydiff_get_scratch(self._ctx, *(ctypes.byref(x) for x in p)))
        U, N, nmax = self.units, self.budget, self.budget + self.max_block
        mk = lambda ptr, shape, ts: torch.as_tensor(_DevArray(ptr.value, shape, ts), device=self.device)
        return {"scores": mk(p[0], (U, nmax), "<f4"), "kept_idx": mk(p[1], (U, N), "<i4"),
                "first_evicted": mk(p[2], (U,), "<i4"), "status": mk(p[3], (1,), "<i4")}

    def positions(self):
        """``keydiff_get_positions`` (slot reuse only): (view of pos [U, N] int32, next position)."""
        p, nxt = ctypes.c_void_p(), ctypes.c_longlong()
        _check(self._lib.keydiff_get_positions(self._ctx, ctypes.byref(p), ctypes.byref(nxt)))
        return torch.as_tensor(_DevArray(p.value, (self.units, self.budget), "<i4"), device=self.device), nxt.value

    def set_positions(self, pos, length: int, next_pos: int, stream: torch.cuda.Stream | None = None):
        """``keydiff_set_positions`` (slot reuse only): resume from a restored cache whose slot -> token position
        map is ``pos`` (int32 CUDA tensor [U, N]; None = identity)."""
        if pos is not None:
            if pos.dtype != torch.int32 or not pos.is_cuda or not pos.is_contiguous() or pos.numel() != self.units * self.budget:
                raise KeyDiffError(KEYDIFF_ERR_INVALID_ARG, "pos: need a contiguous int32 CUDA tensor [U, N]")
        st = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        _check(self._lib.keydiff_set_positions(self._ctx, pos.data_ptr() if pos is not None else None, length, next_pos, st))

    def moved_rows(self) -> int:
        """Cumulative count of kept rows that changed position (synchronises the device)."""
        p = ctypes.c_void_p()
        _check(self._lib.keydiff_get_moved_rows(self._ctx, ctypes.byref(p)))
        t = torch.as_tensor(_DevArray(p.value, (1,), "<i8"), device=self.device)
        return int(t.item())

    def launch_info(self):
        a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check(self._lib.keydiff_get_launch_info(self._ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
        return {"path": a.value, "launches_per_step": b.value, "cluster_size": c.value}

    def close(self):
        if self._ctx:
            self._lib.keydiff_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def evict_static(k_cache, v_cache, new_k, new_v, length: int, stream: torch.cuda.Stream | None = None,
                 eps: float = 0.0) -> int:
    """``keydiff_evict_static``: the eviction step without any device allocation, for callers that
    may not call cudaMalloc (a server whose memory pool owns the GPU, a plugin that only receives
    tensors).  Scratch is a 16 MiB array inside the library, shared by all calls on the device, so
    calls must not overlap on the GPU.  Tensors are bf16 CUDA tensors [units, rows, 128]; ``length``
    is the current cache length.  Returns the new length; raises KeyDiffError (TOO_LARGE) if the
    step needs more than the built-in scratch."""
    lib = load_library()
    U, N, d = k_cache.shape
    B = new_k.shape[1]
    for t in (k_cache, v_cache, new_k, new_v):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
            raise KeyDiffError(KEYDIFF_ERR_INVALID_ARG, "need contiguous bf16 CUDA tensors")
    assert v_cache.shape == k_cache.shape and new_k.shape == (U, B, d) and new_v.shape == (U, B, d)
    st = (stream or torch.cuda.current_stream(k_cache.device)).cuda_stream
    with torch.cuda.device(k_cache.device):   # the library looks the scratch up for the current device
        _check(lib.keydiff_evict_static(k_cache.data_ptr(), v_cache.data_ptr(), new_k.data_ptr(), new_v.data_ptr(),
                                        length, N, B, U, d, eps, st))
    return min(N, length + B)


def selftest_bounded_wait(polls: int = 1000, device=None) -> int:
    """``keydiff_selftest_bounded_wait``: runs the library's bounded wait on a barrier nothing completes and
    returns the status word it leaves (KEYDIFF_ERR_TIMEOUT when failure detection works)."""
    lib = load_library()
    dev = torch.device("cuda", torch.cuda.current_device() if device is None else device)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(lib.keydiff_selftest_bounded_wait(status.data_ptr(), polls, torch.cuda.current_stream(dev).cuda_stream))
        torch.cuda.synchronize(dev)
    return int(status.item())


def debug_fail_alloc(nth: int):
    """``keydiff_debug_fail_alloc``: make the nth device allocation of the next ``keydiff_create`` fail."""
    _check(load_library().keydiff_debug_fail_alloc(nth))
