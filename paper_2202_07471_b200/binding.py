"""Thin ctypes binding of libsquant.so (argument marshalling only; all work runs in the CUDA library).

Function names mirror include/squant.h.  Device-pointer entry points take torch CUDA tensors,
the host entry point takes torch CPU tensors (pinned memory gives full copy speed).
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

MODE_E, MODE_K, MODE_C = 1, 2, 4
MODE_EKC = MODE_E | MODE_K | MODE_C
FLAG_NARROW_RANGE = 1
FLAG_PACK_INT4 = 2

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsquant.so")

NOALLOC_MAX_CTAS = 32768

EXPORTS = ("squant_quantize_layer", "squant_quantize_layer_noalloc", "squant_quantize_model", "squant_quantize_model_host",
           "squant_plan_info", "squant_selfcheck_division", "squant_device_status", "squant_launch_count", "squant_strerror", "squant_last_cuda_error",
           "squant_shutdown", "squant_debug_set_status", "squant_debug_wait_expires", "squant_debug_violations")


class SquantError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"squant error {code}: {text}")
        self.code = code


class Options(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int32), ("mode", ctypes.c_uint32), ("flags", ctypes.c_uint32)]


class Layer(ctypes.Structure):
    _fields_ = [("w", ctypes.c_void_p), ("cout", ctypes.c_int32), ("cin", ctypes.c_int32),
                ("kh", ctypes.c_int32), ("kw", ctypes.c_int32), ("codes", ctypes.c_void_p),
                ("scales", ctypes.c_void_p), ("kernel_err", ctypes.c_void_p),
                ("channel_err", ctypes.c_void_p), ("dequant", ctypes.c_void_p), ("dequant_bf16", ctypes.c_void_p),
                ("scales_in", ctypes.c_void_p)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libsquant.so; there is no fallback implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2202_07471_b200.build` "
            "(needs nvcc); this package has no CPU or PyTorch fallback")
    lib = ctypes.CDLL(LIB_PATH)
    lp, op, vp, i32p = ctypes.POINTER(Layer), ctypes.POINTER(Options), ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)
    lib.squant_quantize_layer.argtypes = [lp, op, vp]
    lib.squant_quantize_layer_noalloc.argtypes = [lp, op, vp]
    lib.squant_quantize_model.argtypes = [lp, ctypes.c_int32, op, vp]
    lib.squant_quantize_model_host.argtypes = [lp, ctypes.c_int32, op, vp]
    lib.squant_plan_info.argtypes = [lp, ctypes.c_int32, op, i32p, i32p, i32p]
    lib.squant_selfcheck_division.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, vp]
    for f in ("squant_quantize_layer", "squant_quantize_layer_noalloc", "squant_quantize_model", "squant_quantize_model_host",
              "squant_plan_info", "squant_selfcheck_division", "squant_device_status", "squant_shutdown"):
        getattr(lib, f).restype = ctypes.c_int
    lib.squant_debug_violations.argtypes = [i32p, i32p]
    lib.squant_debug_violations.restype = ctypes.c_int
    lib.squant_debug_set_status.argtypes = [ctypes.c_int]
    lib.squant_debug_set_status.restype = ctypes.c_int
    lib.squant_debug_wait_expires.argtypes = [ctypes.c_int32, vp]
    lib.squant_debug_wait_expires.restype = ctypes.c_int
    lib.squant_launch_count.restype = ctypes.c_int64
    lib.squant_strerror.restype = ctypes.c_char_p
    lib.squant_strerror.argtypes = [ctypes.c_int]
    lib.squant_last_cuda_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _check(rc: int) -> None:
    if rc != 0:
        lib = load_library()
        text = lib.squant_strerror(rc).decode()
        extra = lib.squant_last_cuda_error().decode()
        raise SquantError(rc, text + (f" [{extra}]" if extra and rc == -7 else ""))


@dataclass
class LayerBuffers:
    """Input and output tensors of one layer (all on one device, or all on the host)."""
    w: torch.Tensor
    codes: torch.Tensor
    scales: torch.Tensor
    kernel_err: Optional[torch.Tensor]
    channel_err: Optional[torch.Tensor]
    dequant: Optional[torch.Tensor] = None     # fp32 code * scale, shape of the weights
    scales_in: Optional[torch.Tensor] = None   # fp32 [cout] caller-supplied scales (None: absmax scales)
    dequant_bf16: Optional[torch.Tensor] = None   # bfloat16 code * scale, shape of the weights


def alloc_outputs(w: torch.Tensor, kernel_err: bool = True, channel_err: bool = True,
                  pin: bool = False, pack_int4: bool = False, dequant: bool = False,
                  dequant_bf16: bool = False) -> LayerBuffers:
    """Allocate output tensors next to `w` ([cout, cin, kh, kw], [cout, cin, k] or [cout, cin]).
    With pack_int4 the codes tensor is [cout, ceil(cin*kh*kw / 2)] (for FLAG_PACK_INT4)."""
    if w.dtype != torch.float32 or not w.is_contiguous() or w.dim() < 2:
        raise ValueError("weights must be a contiguous fp32 tensor [cout, cin, ...]")
    kw = dict(device=w.device)
    if pin and not w.is_cuda:
        kw["pin_memory"] = True
    m, n = w.shape[0], w.shape[1]
    cshape = (m, (w[0].numel() + 1) // 2) if pack_int4 else w.shape
    return LayerBuffers(
        w, torch.empty(cshape, dtype=torch.int8, **kw), torch.empty(m, dtype=torch.float32, **kw),
        torch.empty((m, n), dtype=torch.float32, **kw) if kernel_err else None,
        torch.empty(m, dtype=torch.float32, **kw) if channel_err else None,
        torch.empty(w.shape, dtype=torch.float32, **kw) if dequant else None, None,
        torch.empty(w.shape, dtype=torch.bfloat16, **kw) if dequant_bf16 else None)


def _descriptor(b: LayerBuffers) -> Layer:
    w = b.w
    m, n = int(w.shape[0]), int(w.shape[1])
    if w.dim() == 4:
        kh, kw = int(w.shape[2]), int(w.shape[3])
    elif w.dim() == 3:
        kh, kw = int(w.shape[2]), 1
    elif w.dim() == 2:
        kh, kw = 1, 1
    else:
        raise ValueError("weights must be [cout, cin], [cout, cin, k] or [cout, cin, kh, kw]")
    ptr = lambda t: t.data_ptr() if t is not None else None
    if b.scales_in is not None and (b.scales_in.dtype != torch.float32 or b.scales_in.numel() != m or not b.scales_in.is_contiguous()
                                    or b.scales_in.device != w.device):
        raise ValueError("scales_in must be a contiguous fp32 tensor [cout] next to the weights")
    return Layer(ptr(w), m, n, kh, kw, ptr(b.codes), ptr(b.scales), ptr(b.kernel_err), ptr(b.channel_err), ptr(b.dequant),
                 ptr(b.dequant_bf16), ptr(b.scales_in))


def _options(bits: int, mode: int, flags: int) -> Options:
    return Options(int(bits), int(mode), int(flags))


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


class ModelCall:
    """Descriptors of a fixed set of layers, marshalled once and reusable across calls."""

    def __init__(self, layers: Sequence[LayerBuffers], bits: int = 4, mode: int = MODE_EKC,
                 flags: int = FLAG_NARROW_RANGE):
        self.buffers: List[LayerBuffers] = list(layers)
        self.n = len(self.buffers)
        self.array = (Layer * max(1, self.n))(*[_descriptor(b) for b in self.buffers])
        self.opt = _options(bits, mode, flags)
        self.on_device = bool(self.buffers and self.buffers[0].w.is_cuda)

    def run(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        lib = load_library()
        fn = lib.squant_quantize_model if self.on_device else lib.squant_quantize_model_host
        _check(fn(self.array, self.n, ctypes.byref(self.opt), _stream_handle(stream)))


def squant_quantize_model(layers: Sequence[LayerBuffers], bits: int = 4, mode: int = MODE_EKC,
                          flags: int = FLAG_NARROW_RANGE,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
    """Quantize all layers (device tensors) in one grouped launch on `stream`."""
    call = ModelCall(layers, bits, mode, flags)
    if call.n and not call.on_device:
        raise ValueError("squant_quantize_model needs CUDA tensors; use squant_quantize_model_host")
    call.run(stream)


def squant_quantize_model_host(layers: Sequence[LayerBuffers], bits: int = 4, mode: int = MODE_EKC,
                               flags: int = FLAG_NARROW_RANGE,
                               stream: Optional[torch.cuda.Stream] = None) -> None:
    """Quantize all layers given as host tensors; returns when the outputs are in host memory."""
    call = ModelCall(layers, bits, mode, flags)
    if call.n and call.on_device:
        raise ValueError("squant_quantize_model_host needs CPU tensors")
    call.run(stream)


def squant_quantize_layer(w: torch.Tensor, bits: int = 4, mode: int = MODE_EKC,
                          flags: int = FLAG_NARROW_RANGE,
                          stream: Optional[torch.cuda.Stream] = None) -> LayerBuffers:
    """Quantize one layer held in a CUDA tensor; allocates and returns its outputs."""
    if not w.is_cuda:
        raise ValueError("squant_quantize_layer needs a CUDA tensor")
    b = alloc_outputs(w)
    d = _descriptor(b)
    opt = _options(bits, mode, flags)
    _check(load_library().squant_quantize_layer(ctypes.byref(d), ctypes.byref(opt), _stream_handle(stream)))
    return b


def squant_quantize_layer_noalloc(buffers: LayerBuffers, bits: int = 4, mode: int = MODE_EKC,
                                  flags: int = FLAG_NARROW_RANGE,
                                  stream: Optional[torch.cuda.Stream] = None) -> None:
    """Quantize one layer into caller-provided CUDA tensors without any device allocation.

    For callers that must not allocate GPU memory while running (a framework pool owns the
    device, or the allocation's device-wide synchronisation is not acceptable): the launch table
    lives in a fixed array inside the library.  One layer per call, at most NOALLOC_MAX_CTAS
    thread blocks (SquantError code -9 beyond that), and calls whose GPU work may overlap must be
    serialised by the caller because they share that array.  This wrapper itself creates no
    tensors; results equal squant_quantize_layer bit for bit."""
    if not buffers.w.is_cuda:
        raise ValueError("squant_quantize_layer_noalloc needs CUDA tensors")
    d = _descriptor(buffers)
    opt = _options(bits, mode, flags)
    _check(load_library().squant_quantize_layer_noalloc(ctypes.byref(d), ctypes.byref(opt),
                                                        _stream_handle(stream)))


def squant_plan_info(shapes: Sequence[Sequence[int]], bits: int = 4, mode: int = MODE_EKC,
                     flags: int = FLAG_NARROW_RANGE) -> dict:
    """Launch geometry for layers of the given [cout, cin, kh, kw] shapes (no GPU needed)."""
    arr = (Layer * max(1, len(shapes)))(*[Layer(None, int(s[0]), int(s[1]), int(s[2]), int(s[3]),
                                                None, None, None, None, None, None, None) for s in shapes])
    opt = _options(bits, mode, flags)
    g, t, s = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().squant_plan_info(arr, len(shapes), ctypes.byref(opt), ctypes.byref(g),
                                           ctypes.byref(t), ctypes.byref(s)))
    return {"grid_ctas": g.value, "cta_threads": t.value, "dynamic_smem_bytes": s.value}


def squant_selfcheck_division(scales, bits: int = 4):
    """Exhaustive device check of the reciprocal-based division for the given scales (numpy fp32).
    Returns a numpy uint64 array of mismatch counts (must be all zero)."""
    import numpy as np
    sc = np.ascontiguousarray(scales, dtype=np.float32)
    out = np.zeros(sc.size, dtype=np.uint64)
    _check(load_library().squant_selfcheck_division(sc.ctypes.data_as(ctypes.c_void_p), sc.size, int(bits),
                                                   out.ctypes.data_as(ctypes.c_void_p), _stream_handle(None)))
    return out


def squant_device_status() -> None:
    """Synchronise the current device; raise SquantError(-10) if a kernel gave up a bounded wait."""
    _check(load_library().squant_device_status())


def use_library(path: Optional[str]) -> None:
    """Switch to another build of the library (the checked one, for tests); None: the regular one."""
    global _lib, LIB_PATH
    _lib = None
    LIB_PATH = path if path is not None else os.path.join(_HERE, "libsquant.so")


def squant_debug_violations():
    """(checked build?, failed checks since the last call, site of the first)."""
    n, site = ctypes.c_int32(), ctypes.c_int32()
    rc = load_library().squant_debug_violations(ctypes.byref(n), ctypes.byref(site))
    if rc < 0:
        _check(rc)
    return bool(rc), n.value, site.value


def squant_debug_set_status(value: int) -> None:
    """Test hook: write the device status word as a kernel that gave up a wait would."""
    _check(load_library().squant_debug_set_status(int(value)))


def squant_debug_wait_expires(max_polls: int = 64, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Test hook: one warp waits (at most max_polls polls) on a barrier nobody arrives at."""
    _check(load_library().squant_debug_wait_expires(int(max_polls), _stream_handle(stream)))


def squant_launch_count() -> int:
    return int(load_library().squant_launch_count())


def squant_shutdown() -> None:
    _check(load_library().squant_shutdown())
