"""The C-ABI library builds, loads without a GPU and exports every symbol include/seg.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2403_11204_b200 import build, binding
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "seg.h")).read()
    return sorted(set(re.findall(r"SEG_API\s+[\w\s\*]+?\b(seg_\w+)\s*\(", text)))


def test_header_declares_the_five_calls():
    names = declared_symbols()
    for n in ("seg_create", "seg_gen_labels", "seg_train_step", "seg_forward", "seg_destroy"):
        assert n in names


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2403_11204_b200 import binding
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
        assert n in binding.EXPORTS, f"{n} has no ctypes signature"
    assert sorted(binding.EXPORTS) == names


def test_status_strings_and_argument_errors_need_no_gpu(lib):
    from paper_2403_11204_b200 import binding
    assert lib.seg_status_string(0) == b"ok"
    assert b"unknown" in lib.seg_status_string(99)
    assert b"sm_100a" in lib.seg_build_info()
    h = ctypes.c_void_p()
    assert lib.seg_create(None, ctypes.byref(h)) == 1               # invalid argument
    cfg = binding.seg_config()
    w = (ctypes.c_int32 * 3)(4, 3, 2)
    cfg.n_layers, cfg.widths, cfg.n_classes, cfg.max_batch = 0, w, 2, 4
    assert lib.seg_create(ctypes.byref(cfg), ctypes.byref(h)) == 2  # shape: zero layers
    cfg.n_layers, cfg.is_final = 2, 1
    cfg.n_classes = 5                                               # final width 2 != 5 classes
    assert lib.seg_create(ctypes.byref(cfg), ctypes.byref(h)) == 2
    assert lib.seg_destroy(None) == 1
    assert lib.seg_train_step(None, None, None, 1, None, None) == 1


def test_product_path_fails_loudly_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2403_11204_b200 import binding
    cfg = binding.seg_config()
    w = (ctypes.c_int32 * 3)(4, 3, 2)
    cfg.n_layers, cfg.widths, cfg.n_classes, cfg.max_batch = 2, w, 2, 4
    h = ctypes.c_void_p()
    assert lib.seg_create(ctypes.byref(cfg), ctypes.byref(h)) == 8  # no usable device, no fallback
    assert not h.value
    with pytest.raises(RuntimeError):
        binding.Segment([4, 3, 2], 2, False)
