"""squant_quantize_layer_noalloc: the entry point for callers that may not allocate GPU memory
while they run (a framework's memory pool owns the device, or cudaMalloc's device-wide
synchronisation is unaffordable).  Its launch table sits in a fixed array inside the library
instead of cudaMalloc'ed memory, so everything it produces must equal what
squant_quantize_layer produces, bit for bit, on every call - including a second call that
reuses the same array with a different layer.

Collected last on purpose (file name): a failure here cannot hide results of other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2202_07471_b200 as sq
from paper_2202_07471_b200 import binding, workloads as W


def test_layer_beyond_the_fixed_table_is_rejected_without_a_gpu():
    """More thread blocks than SQUANT_NOALLOC_MAX_CTAS: a clear error before any CUDA call."""
    lib = sq.load_library()
    m = sq.NOALLOC_MAX_CTAS + 1                      # channels of 18432 weights: one block each
    assert sq.squant_plan_info([(m, 2048, 3, 3)])["grid_ctas"] == m
    layer = binding.Layer(256, m, 2048, 3, 3, 256, 256, None, None, None, None, None)   # never dereferenced
    opt = binding.Options(4, sq.MODE_EKC, sq.FLAG_NARROW_RANGE)
    rc = lib.squant_quantize_layer_noalloc(ctypes.byref(layer), ctypes.byref(opt), None)
    assert rc == -9
    assert "SQUANT_NOALLOC_MAX_CTAS" in lib.squant_strerror(rc).decode()
    assert lib.squant_quantize_layer_noalloc(None, ctypes.byref(opt), None) == -1


def _same(a: sq.LayerBuffers, b: sq.LayerBuffers) -> bool:
    # bit-exact, as in the parity tests: integer codes and raw float words
    return (torch.equal(a.codes, b.codes)
            and torch.equal(a.scales.view(torch.int32), b.scales.view(torch.int32))
            and torch.equal(a.kernel_err.view(torch.int32), b.kernel_err.view(torch.int32))
            and torch.equal(a.channel_err.view(torch.int32), b.channel_err.view(torch.int32)))


@pytest.mark.gpu
def test_noalloc_matches_regular_entry_point_on_consecutive_calls():
    shapes = [(96, 128, 3, 3), (300, 1000, 1, 1), (40, 2048, 3, 3), (96, 128, 3, 3)]
    for bits in (4, 8):
        for i, shp in enumerate(shapes):                 # back-to-back calls share the table
            w = torch.from_numpy(W.random_layer(shp, seed=31 + i)).cuda()
            want = sq.squant_quantize_layer(w, bits=bits)
            got = sq.alloc_outputs(w)                    # outputs allocated by the caller, up front
            got.codes.fill_(-128)
            got.scales.fill_(float("nan"))
            got.kernel_err.fill_(float("nan"))
            got.channel_err.fill_(float("nan"))
            n0 = sq.squant_launch_count()
            sq.squant_quantize_layer_noalloc(got, bits=bits)
            sq.squant_quantize_layer_noalloc(got, bits=bits)      # twice in a row, same stream
            torch.cuda.synchronize()
            assert sq.squant_launch_count() == n0 + 2
            assert _same(got, want), f"shape {shp} bits {bits}"
            ref = oracle.quantize_layer(w.cpu().numpy(), bits=bits)      # and with the CPU checker directly
            assert np.array_equal(got.codes.cpu().numpy(), ref.codes) and np.array_equal(got.scales.cpu().numpy(), ref.scales)
            assert np.array_equal(got.kernel_err.cpu().numpy(), ref.kernel_err)
            assert np.array_equal(got.channel_err.cpu().numpy(), ref.channel_err)


@pytest.mark.gpu
def test_noalloc_refuses_a_stream_that_is_being_captured():
    """The table upload reads a host image that the next call rewrites, so a captured copy would
    replay someone else's table: the call is refused before anything is enqueued, and the same
    call works again on the same stream once the capture is over."""
    w = torch.from_numpy(W.random_layer((32, 64, 3, 3), seed=5)).cuda()
    got = sq.alloc_outputs(w)
    sq.squant_quantize_layer_noalloc(got, bits=4)        # first call on the device: outside any capture
    torch.cuda.synchronize()
    want = got.codes.clone()
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    n0 = sq.squant_launch_count()
    with torch.cuda.graph(g, stream=s):
        with pytest.raises(sq.SquantError) as ei:
            sq.squant_quantize_layer_noalloc(got, bits=4, stream=torch.cuda.current_stream())
    assert ei.value.code == -11 and sq.squant_launch_count() == n0
    got.codes.fill_(-128)
    sq.squant_quantize_layer_noalloc(got, bits=4, stream=s)
    s.synchronize()
    assert torch.equal(got.codes, want)
