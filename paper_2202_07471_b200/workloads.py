"""Seeded synthetic weight generators and layer-shape tables.

This module only produces INPUTS (layer shapes and fp32 weight values).  It holds
none of the quantization method's arithmetic and is the one piece of code that both
the CUDA path's tests and the CPU checker's tests draw their data from.

Random numbers come from a counter-based generator built on the published
splitmix64 finaliser (Steele, Lea, Flood 2014): value i of a stream is
mix(stream_key + (i + 1) * GOLDEN).  Because it is counter based, any slice of any
layer can be generated independently and reproducibly, whatever numpy version runs.

The model-shaped workloads stand in for the trained ImageNet CNNs the paper
quantizes (its Table 3 lists ResNet18 with 21 layers and ResNet50 with 54 layers):
only the public layer SHAPES are used, filled with seeded synthetic values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Iterator, List, Sequence, Tuple

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK = (1 << 64) - 1


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on a uint64 array (wrapping arithmetic)."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _mix64_scalar(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def stream_key(*parts: int) -> int:
    """Derive a 64-bit stream key from integers (config id, seed, layer, substream...)."""
    k = 0x243F6A8885A308D3
    for p in parts:
        k = _mix64_scalar(k ^ _mix64_scalar((int(p) + 0x9E3779B97F4A7C15) & _MASK))
    return k


def raw_u64(key: int, start: int, count: int) -> np.ndarray:
    """Values start .. start+count-1 of stream `key` as uint64."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        return _mix64(np.uint64(key) + idx * _GOLDEN)


def uniform01(key: int, start: int, count: int) -> np.ndarray:
    """float64 uniforms strictly inside (0, 1)."""
    u = raw_u64(key, start, count) >> np.uint64(11)
    return (u.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(key: int, start: int, count: int) -> np.ndarray:
    """Standard normals (float64) by Box-Muller; normal i uses uniforms 2i and 2i+1."""
    u = uniform01(key, 2 * start, 2 * count)
    return np.sqrt(-2.0 * np.log(u[0::2])) * np.cos((2.0 * math.pi) * u[1::2])


# --------------------------------------------------------------------------------------
# layer shape tables  (cout, cin, kh, kw); cin is the per-kernel input-channel count, so a
# depthwise conv has cin = 1.
# --------------------------------------------------------------------------------------
Shape = Tuple[int, int, int, int]


def single_conv_shapes() -> List[Shape]:
    return [(64, 64, 3, 3)]


def resnet18_shapes() -> List[Shape]:
    s: List[Shape] = [(64, 3, 7, 7)]
    s += [(64, 64, 3, 3)] * 4
    cin = 64
    for w in (128, 256, 512):
        s += [(w, cin, 3, 3)] + [(w, w, 3, 3)] * 3 + [(w, cin, 1, 1)]
        cin = w
    s.append((1000, 512, 1, 1))
    return s


def resnet50_shapes() -> List[Shape]:
    s: List[Shape] = [(64, 3, 7, 7)]
    cin = 64
    for w, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            s += [(w, cin, 1, 1), (w, w, 3, 3), (4 * w, w, 1, 1)]
            if b == 0:
                s.append((4 * w, cin, 1, 1))
            cin = 4 * w
    s.append((1000, 2048, 1, 1))
    return s


def mobilenetv2_shapes() -> List[Shape]:
    s: List[Shape] = [(32, 3, 3, 3)]
    cin = 32
    for t, c, n in ((1, 16, 1), (6, 24, 2), (6, 32, 3), (6, 64, 4), (6, 96, 3), (6, 160, 3), (6, 320, 1)):
        for _ in range(n):
            hidden = t * cin
            if t != 1:
                s.append((hidden, cin, 1, 1))
            s.append((hidden, 1, 3, 3))
            s.append((c, hidden, 1, 1))
            cin = c
    s.append((1280, 320, 1, 1))
    s.append((1000, 1280, 1, 1))
    return s


def mixed_kernel_shapes() -> List[Shape]:
    """A synthetic family (not a published architecture) with the kernel shapes of
    Inception / SqueezeNext / ShuffleNet style networks: factorised 1x7 / 7x1 / 1x3 / 3x1
    convolutions, 5x5 and 3x3 convolutions, grouped convolutions (few input channels per kernel
    group), pointwise layers and a classifier; 64 layers."""
    s: List[Shape] = [(32, 3, 3, 3), (32, 32, 3, 3), (64, 32, 3, 3), (80, 64, 1, 1), (192, 80, 3, 3)]
    for c in (192, 256, 288):
        s += [(64, c, 1, 1), (48, c, 1, 1), (64, 48, 5, 5), (64, c, 1, 1), (96, 64, 3, 3), (96, 96, 3, 3)]
    for c in (128, 160, 192):
        s += [(192, 768, 1, 1), (c, 768, 1, 1), (c, c, 1, 7), (192, c, 7, 1), (c, c, 7, 1), (192, c, 1, 7)]
    s += [(320, 1280, 1, 1), (384, 1280, 1, 1), (384, 384, 1, 3), (384, 384, 3, 1), (448, 1280, 1, 1), (384, 448, 3, 3)]
    for c, g in ((240, 3), (480, 4), (960, 8)):          # grouped: cin per group = c / g
        s += [(c, c // g, 1, 1), (c, 1, 3, 3), (c, c // g, 1, 1), (c // 2, c // (2 * g), 3, 1), (c // 2, c // (2 * g), 1, 3)]
    s += [(1000, 2048, 1, 1), (1001, 1537, 1, 1)]
    return s


def large_layer_shapes() -> List[Shape]:
    return [(2048, 2048, 3, 3)] * 8


@dataclass(frozen=True)
class Workload:
    """A named list of layers plus the value recipe used to fill them."""
    name: str
    config_id: int
    shapes: Tuple[Shape, ...]
    recipe: str           # 'normal' | 'normal_laplace' | 'student_t4' | 'normal_chanscale'
    bits: Tuple[int, ...]

    @property
    def n_weights(self) -> int:
        return sum(m * n * kh * kw for m, n, kh, kw in self.shapes)

    @property
    def n_channels(self) -> int:
        return sum(m for m, _, _, _ in self.shapes)


WORKLOADS = {
    "single_conv": Workload("single_conv", 1, tuple(single_conv_shapes()), "normal", (4,)),
    "resnet18": Workload("resnet18", 2, tuple(resnet18_shapes()), "normal_laplace", (4,)),
    "resnet50": Workload("resnet50", 3, tuple(resnet50_shapes()), "student_t4", (4, 6)),
    "mobilenetv2": Workload("mobilenetv2", 4, tuple(mobilenetv2_shapes()), "normal", (4,)),
    "mixed_kernels": Workload("mixed_kernels", 6, tuple(mixed_kernel_shapes()), "normal_laplace", (4,)),
    "large_layer": Workload("large_layer", 5, tuple(large_layer_shapes()), "normal_chanscale", (4,)),
}


def _fan_in_std(shape: Shape) -> float:
    _, n, kh, kw = shape
    return math.sqrt(2.0 / (n * kh * kw))


def _fill(recipe: str, key: int, start: int, count: int, std: float) -> np.ndarray:
    """float64 values start..start+count-1 of one layer's value stream."""
    if recipe in ("normal", "normal_chanscale"):
        return normal(key, start, count) * std
    if recipe == "normal_laplace":
        base = normal(key, start, count) * std
        pick = uniform01(stream_key(key, 1), start, count) < 0.05
        u = uniform01(stream_key(key, 2), start, count) - 0.5
        lap = -(3.0 * std) * np.sign(u) * np.log1p(-2.0 * np.abs(u))
        return np.where(pick, lap, base)
    if recipe == "student_t4":
        z = normal(key, start, count)
        u = uniform01(stream_key(key, 3), 2 * start, 2 * count)
        chi2 = -2.0 * np.log(u[0::2] * u[1::2])          # chi-square with 4 degrees of freedom
        return z / np.sqrt(chi2 / 4.0) * (std / math.sqrt(2.0))
    raise ValueError(f"unknown recipe {recipe!r}")


def _fill_channels(wl: Workload, layer: int, seed: int, c0: int, c1: int, out: np.ndarray,
                   chunk: int) -> None:
    """Write channels c0..c1-1 of one layer into out[(c1-c0) * per_ch] (flat fp32)."""
    m, n, kh, kw = wl.shapes[layer]
    per_ch = n * kh * kw
    key = stream_key(wl.config_id, seed, layer)
    std = _fan_in_std(wl.shapes[layer])
    lo, hi = c0 * per_ch, c1 * per_ch
    for s in range(lo, hi, chunk):
        e = min(hi, s + chunk)
        out[s - lo:e - lo] = _fill(wl.recipe, key, s, e - s, std).astype(np.float32)
    if wl.recipe == "normal_chanscale":
        u = uniform01(stream_key(key, 4), c0, c1 - c0)
        mult = np.exp(math.log(0.5) + u * (math.log(2.0) - math.log(0.5)))
        out.reshape(c1 - c0, per_ch)[...] *= mult.astype(np.float32)[:, None]


def layer_weights(wl: Workload, layer: int, seed: int = 0, *, channels: slice | None = None,
                  chunk: int = 1 << 20, threads: int = 1, out: np.ndarray | None = None) -> np.ndarray:
    """fp32 weights of one layer, shape [cout, cin, kh, kw] (or the selected channel range).

    Values depend only on (workload, layer, seed, position): any channel range, chunk size or
    thread count gives the same numbers.  `out` may be a preallocated fp32 array to fill."""
    m, n, kh, kw = wl.shapes[layer]
    per_ch = n * kh * kw
    c0, c1, _ = (channels or slice(None)).indices(m)
    if out is None:
        out = np.empty((c1 - c0, n, kh, kw), dtype=np.float32)
    flat = out.reshape(-1)
    assert flat.size == (c1 - c0) * per_ch and flat.dtype == np.float32
    threads = max(1, min(int(threads), c1 - c0))
    if threads == 1:
        _fill_channels(wl, layer, seed, c0, c1, flat, chunk)
    else:
        from concurrent.futures import ThreadPoolExecutor
        n_parts = min(c1 - c0, threads * 4)
        edges = [c0 + (c1 - c0) * i // n_parts for i in range(n_parts + 1)]
        with ThreadPoolExecutor(threads) as pool:
            futs = [pool.submit(_fill_channels, wl, layer, seed, a, b,
                                flat[(a - c0) * per_ch:(b - c0) * per_ch], chunk)
                    for a, b in zip(edges[:-1], edges[1:]) if b > a]
            for f in futs:
                f.result()
    return out.reshape(c1 - c0, n, kh, kw)


def iter_layers(wl: Workload, seed: int = 0) -> Iterator[Tuple[int, Shape, np.ndarray]]:
    for i, shp in enumerate(wl.shapes):
        yield i, shp, layer_weights(wl, i, seed)


def random_layer(shape: Sequence[int], seed: int, std: float | None = None) -> np.ndarray:
    """A free-standing N(0, std) layer for shape sweeps (std defaults to fan-in Kaiming)."""
    shape = tuple(int(v) for v in shape)
    count = int(np.prod(shape))
    if std is None:
        std = math.sqrt(2.0 / max(1, count // shape[0]))
    key = stream_key(99, seed, *shape)
    return (normal(key, 0, count) * std).astype(np.float32).reshape(shape)
