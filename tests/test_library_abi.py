"""Host-side checks that need no GPU: the C-ABI library builds, loads, and exports every symbol
include/keydiff.h declares; host-detectable errors are reported without any device work."""
import ctypes
import os
import re

import pytest
import torch

from paper_2504_15364_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load_library()


def test_header_symbols_are_exported(lib):
    header = open(os.path.join(ROOT, "include", "keydiff.h")).read()
    declared = set(re.findall(r"KEYDIFF_API\s+[\w\s\*]+?\b(keydiff_\w+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_strerror_names_every_code(lib):
    texts = {lib.keydiff_strerror(c).decode() for c in range(0, -9, -1)}
    assert len(texts) == 9 and "unknown keydiff status" not in texts
    assert lib.keydiff_strerror(-99).decode() == "unknown keydiff status"


def test_null_and_bad_config_rejected_before_any_device_work(lib):
    out = ctypes.c_void_p()
    assert lib.keydiff_create(None, ctypes.byref(out)) == binding.KEYDIFF_ERR_INVALID_ARG
    cfg = binding.keydiff_config(1, 1, 8, 128, 512, 128, binding.KEYDIFF_BF16, 0, 0.0, 0)
    assert lib.keydiff_create(ctypes.byref(cfg), None) == binding.KEYDIFF_ERR_INVALID_ARG
    for field, bad in [("n_layers", 0), ("budget", 0), ("max_block", -1), ("device", -1), ("path", 7),
                       ("anchor_mode", 2), ("recent_window", -1), ("recent_window", 513), ("compaction", 2)]:
        c = binding.keydiff_config(1, 1, 8, 128, 512, 128, binding.KEYDIFF_BF16, 0, 0.0, 0)
        setattr(c, field, bad)
        assert lib.keydiff_create(ctypes.byref(c), ctypes.byref(out)) == binding.KEYDIFF_ERR_INVALID_ARG, field
    c = binding.keydiff_config(1, 1, 8, 64, 512, 128, binding.KEYDIFF_BF16, 0, 0.0, 0)      # head_dim 64
    assert lib.keydiff_create(ctypes.byref(c), ctypes.byref(out)) == binding.KEYDIFF_ERR_UNSUPPORTED
    c = binding.keydiff_config(1, 1, 8, 128, 512, 128, 5, 0, 0.0, 0)                          # dtype
    assert lib.keydiff_create(ctypes.byref(c), ctypes.byref(out)) == binding.KEYDIFF_ERR_UNSUPPORTED
    assert lib.keydiff_destroy(None) == binding.KEYDIFF_OK
    assert lib.keydiff_get_len(None, None) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_get_positions(None, None, None) == binding.KEYDIFF_ERR_INVALID_ARG
    assert lib.keydiff_evict(None, None, None, None, None, 1, 1, 1, 128, None) == binding.KEYDIFF_ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_create_fails_loudly_without_a_gpu(lib):
    # no CPU fallback: without a CUDA device the product path raises
    with pytest.raises(binding.KeyDiffError) as ei:
        binding.KeyDiff(1, 1, 8, 128, 512, 128)
    assert ei.value.code in (binding.KEYDIFF_ERR_CUDA, binding.KEYDIFF_ERR_UNSUPPORTED)
