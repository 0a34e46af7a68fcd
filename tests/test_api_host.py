"""Host-side checks that need no GPU: the library loads, exports what include/squant.h declares,
validates arguments and plans launches."""
import ctypes
import os
import re

import pytest

import paper_2202_07471_b200 as sq
from paper_2202_07471_b200 import binding, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = sq.load_library()
    header = open(os.path.join(ROOT, "include", "squant.h")).read()
    declared = set(re.findall(r"\b(squant_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in squant.h but not exported"
    assert declared == set(binding.EXPORTS)


def test_strerror_covers_all_codes():
    lib = sq.load_library()
    texts = {lib.squant_strerror(c).decode() for c in range(0, -12, -1)}
    assert len(texts) == 12 and all(texts)
    assert "unknown" in lib.squant_strerror(-99).decode()


def _info(shapes, **kw):
    return sq.squant_plan_info(shapes, **kw)


def test_plan_geometry_for_the_five_configs():
    for name, wl in W.WORKLOADS.items():
        info = _info(wl.shapes)
        assert info["cta_threads"] == 256
        assert 0 < info["dynamic_smem_bytes"] <= 232448
        assert info["grid_ctas"] >= 1
    # one CTA per output channel for the large layers
    assert _info(W.WORKLOADS["large_layer"].shapes)["grid_ctas"] == 8 * 2048
    # small channels share a CTA: 8 warps, one channel each
    assert _info([(64, 64, 3, 3)])["grid_ctas"] == 8   # 64 channels, 8 one-warp groups per 256-thread block
    assert _info([(33, 7, 3, 3)])["grid_ctas"] == 5
    assert _info([(600, 1, 3, 3)])["grid_ctas"] == 3   # depthwise: a whole channel per thread, 256 per block


@pytest.mark.parametrize("shape,kw,code", [
    ((0, 3, 3, 3), {}, -2), ((4, -1, 3, 3), {}, -2), ((4, 3, 0, 3), {}, -2),
    ((4, 3, 3, 3), {"bits": 1}, -3), ((4, 3, 3, 3), {"bits": 9}, -3),
    ((4, 3, 3, 3), {"mode": 2}, -4), ((4, 3, 3, 3), {"mode": 8 | 1}, -4),
    ((4, 3, 3, 3), {"mode": 16 | 1}, -4), ((4, 3, 3, 3), {"flags": 16}, -4),
    ((4, 3, 3, 3), {"bits": 6, "flags": 3}, -3),
    ((4, 70000, 1, 1), {}, -6), ((4, 8000, 3, 3), {}, -6),
])
def test_invalid_arguments_are_rejected(shape, kw, code):
    with pytest.raises(sq.SquantError) as ei:
        _info([shape], **kw)
    assert ei.value.code == code


def test_valid_edge_arguments():
    assert _info([], bits=4)["grid_ctas"] == 0
    assert _info([(4, 300, 1, 1)], mode=1 | 4)["grid_ctas"] >= 1      # E|C ablation mode
    assert _info([(4, 30, 3, 3)], mode=1 | 4)["grid_ctas"] >= 1
    assert _info([(1, 1, 1, 1)], bits=2)["grid_ctas"] == 1
    assert _info([(2, 4000, 3, 3)])["grid_ctas"] == 2


def test_null_pointers_are_rejected_before_any_cuda_call():
    lib = sq.load_library()
    layer = binding.Layer(None, 4, 3, 3, 3, None, None, None, None, None, None, None)
    opt = binding.Options(4, 7, 1)
    assert lib.squant_quantize_layer(ctypes.byref(layer), ctypes.byref(opt), None) == -1
    assert lib.squant_quantize_model(None, 2, ctypes.byref(opt), None) == -1
    assert lib.squant_quantize_model(None, 0, ctypes.byref(opt), None) == 0
    assert lib.squant_quantize_layer(None, ctypes.byref(opt), None) == -1
    layer = binding.Layer(1026, 4, 3, 3, 3, 64, 128, None, None, None, None, None)      # weights not 4-byte aligned
    assert lib.squant_quantize_layer(ctypes.byref(layer), ctypes.byref(opt), None) == -5


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libsquant.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()
