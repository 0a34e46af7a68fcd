"""Input builders for parity tests (inputs only; no quantization arithmetic)."""
import math

import numpy as np

from paper_2202_07471_b200 import workloads as W


def coarse(w: np.ndarray, steps: int = 40, div: int = 8) -> np.ndarray:
    """Snap values to a coarse grid: many equal perturbations and exact halves."""
    return (np.round(w / np.abs(w).max() * steps) / div).astype(np.float32)


def adversarial_layer(shape, seed: int) -> np.ndarray:
    """Random layer with special channels mixed in: all-zero, single non-zero, constant, tiny,
    huge, coarse-grid (ties), duplicated kernels."""
    w = W.random_layer(shape, seed)
    m = shape[0]
    rng = np.random.default_rng(seed)
    kinds = rng.integers(0, 9, size=m)
    for c in range(m):
        k = kinds[c]
        if k == 0:
            w[c] = 0.0
        elif k == 1:
            v = w[c].reshape(-1)[0]
            w[c] = 0.0
            w[c].reshape(-1)[rng.integers(0, w[c].size)] = v if v != 0 else 1.0
        elif k == 2:
            w[c] = np.float32(0.3) * np.float32(rng.choice([-1.0, 1.0]))
        elif k == 3:
            w[c] *= np.float32(2.0 ** -112)          # below the 2^-100 scale floor
        elif k == 4:
            w[c] *= np.float32(2.0 ** rng.integers(-90, 90))
        elif k == 5:
            w[c] = coarse(w[c])
        elif k == 6 and w.shape[1] > 1:
            w[c, 1:] = w[c, :1]                      # every kernel equal: candidate ties in SQuant-C
    return w


SWEEP_SHAPES = []
for K in ((1, 1), (2, 1), (3, 1), (2, 2), (3, 3), (5, 5), (7, 7), (1, 7), (11, 11)):
    for N in (1, 2, 3, 31, 32, 33, 64, 100, 257):
        if N * K[0] * K[1] <= 20000:
            SWEEP_SHAPES.append((5 if N * K[0] * K[1] > 2000 else 19, N, K[0], K[1]))
# channel lengths around every group-size boundary of the launch plan, and wide ones
SWEEP_SHAPES += [(3, 1024, 1, 1), (3, 1025, 1, 1), (3, 2048, 1, 1), (3, 2049, 1, 1), (3, 4099, 1, 1),
                 (2, 8192, 1, 1), (2, 8200, 1, 1), (2, 20011, 1, 1), (2, 1024, 3, 3), (2, 2048, 3, 3),
                 (2, 455, 3, 3), (2, 911, 3, 3), (3, 114, 3, 3), (2, 3000, 3, 3), (40, 7, 3, 3)]


def redo_layer(n: int = 2048, bits: int = 4, seed: int = 3) -> np.ndarray:
    """A [6, n, 3, 3] layer whose channels hold controlled fractions (0, 1 %, 30 %, 49 %, 51 %, all)
    of kernels that a fast 3x3 selection cannot settle: kernels whose weights are all tiny against
    the channel's scale, and kernels whose nine rounding errors have one sign and sum to about 4.
    One weight per channel equals qmax * 2^-5, so the channel's scale is exactly 2^-5."""
    rng = np.random.default_rng(seed)
    qmax = 2 ** (bits - 1) - 1
    s0 = 2.0 ** -5
    fracs = (0.0, 0.01, 0.30, 0.49, 0.51, 1.0)
    w = np.empty((len(fracs), n, 9), dtype=np.float64)
    for c, f in enumerate(fracs):
        x = rng.uniform(-qmax + 0.6, qmax - 0.6, size=(n, 9))           # ordinary kernels
        hard = rng.random(n) < f
        tiny = rng.uniform(-1.0 / 16, 1.0 / 16, size=(n, 9))             # every |x| < 1/8
        sgn = rng.choice([-1.0, 1.0], size=(n, 1))
        big = np.round(rng.uniform(-qmax + 1, qmax - 1, size=(n, 9))) + sgn * rng.uniform(0.42, 0.49, size=(n, 9))
        kind = rng.random(n) < 0.5
        x[hard & kind] = tiny[hard & kind]
        x[hard & ~kind] = big[hard & ~kind]
        x[0, 0] = qmax                                                    # fixes absmax and the scale
        w[c] = x * s0
    return w.reshape(len(fracs), n, 3, 3).astype(np.float32)
