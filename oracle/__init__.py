"""CPU checker for the SQuant solver -- TEST INFRASTRUCTURE, not part of the product path.

Only tests/, the smoke check and the benchmark's CPU-baseline leg may import this package.
It wraps oracle/squant_oracle.c (plain single-threaded C) through ctypes with host numpy
arrays; it shares no code with the CUDA implementation and never imports it.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from typing import Optional

import numpy as np

from . import build as _build

MODE_E, MODE_K, MODE_C = 1, 2, 4
MODE_EKC = MODE_E | MODE_K | MODE_C
FLAG_NARROW_RANGE = 1
FLAG_PACK_INT4 = 2
ONE = 1 << 30
HALF = 1 << 29


class _Options(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int32), ("mode", ctypes.c_uint32), ("flags", ctypes.c_uint32)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.sqo_quantize_layer_scaled.restype = ctypes.c_int
        lib.sqo_quantize_layer_scaled.argtypes = [
            ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            ctypes.POINTER(_Options), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


@dataclass
class OracleResult:
    codes: np.ndarray                      # int8, shape of the weights ([M, ceil(N*K/2)] if packed)
    scales: np.ndarray                     # fp32 [M]
    kernel_err: np.ndarray                 # fp32 [M, N]
    channel_err: np.ndarray                # fp32 [M]
    pert: Optional[np.ndarray] = None      # int32 fixed-point perturbations (2^-30 units)
    flip: Optional[np.ndarray] = None      # uint8: bit0 flipped by SQuant-K, bit1 by SQuant-C
    dequant: Optional[np.ndarray] = None   # fp32 code * scale (what Algorithm 1 returns)
    dequant_bf16: Optional[np.ndarray] = None   # the same as bfloat16 bit patterns (uint16)


def quantize_layer(w: np.ndarray, bits: int = 4, mode: int = MODE_EKC,
                   flags: int = FLAG_NARROW_RANGE, *, details: bool = False,
                   scales_in: Optional[np.ndarray] = None) -> OracleResult:
    """Run the checker on one layer.  `w` is [M, N, kh, kw], [M, N, K] or [M, N] fp32.
    scales_in ([M] fp32) replaces the absmax scales by the caller's (Algorithm 1's input s)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    if w.ndim < 2:
        raise ValueError("weights need at least [M, N]")
    M, N = int(w.shape[0]), int(w.shape[1])
    K = int(np.prod(w.shape[2:])) if w.ndim > 2 else 1
    if flags & FLAG_PACK_INT4:
        codes = np.empty((M, (N * K + 1) // 2), dtype=np.int8)
    else:
        codes = np.empty(w.shape, dtype=np.int8)
    scales = np.empty(M, dtype=np.float32)
    kerr = np.empty((M, N), dtype=np.float32)
    cerr = np.empty(M, dtype=np.float32)
    pert = np.empty(w.shape, dtype=np.int32) if details else None
    flip = np.empty(w.shape, dtype=np.uint8) if details else None
    deq = np.empty(w.shape, dtype=np.float32) if details else None
    deq16 = np.empty(w.shape, dtype=np.uint16) if details else None
    opt = _Options(bits, mode, flags)
    ptr = lambda a: a.ctypes.data_as(ctypes.c_void_p) if a is not None else None
    sin = None
    if scales_in is not None:
        sin = np.ascontiguousarray(scales_in, dtype=np.float32)
        if sin.shape != (M,):
            raise ValueError("scales_in needs one fp32 scale per output channel")
    rc = _load().sqo_quantize_layer_scaled(ptr(w), M, N, K, ctypes.byref(opt), ptr(codes), ptr(scales),
                                           ptr(kerr), ptr(cerr), ptr(pert), ptr(flip), ptr(deq), ptr(sin), ptr(deq16))
    if rc != 0:
        raise ValueError(f"sqo_quantize_layer failed with code {rc}")
    return OracleResult(codes, scales, kerr, cerr, pert, flip, deq, deq16)
