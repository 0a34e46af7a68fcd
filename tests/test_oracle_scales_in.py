"""Pins for the checker's caller-supplied-scale mode.

Algorithm 1 takes the scale vector s as an input and Sec. 2.2 clips round(w / s) to the integer
range; the paper does not say what SQuant-K / SQuant-C do with clipped elements.  The reading
pinned here: a clipped element keeps its saturated code, its perturbation enters every sum, it is
never flipped outward, and when fewer candidates exist than round(|e|) asks for, all are flipped
and the error sums report what is left.  Unit: 2^-30 (ONE = 2^30, HALF = 2^29).
"""
import itertools

import numpy as np
import pytest

import oracle
from oracle import HALF, ONE
from paper_2202_07471_b200 import workloads as W

E, EK, EC, EKC = (oracle.MODE_E, oracle.MODE_E | oracle.MODE_K, oracle.MODE_E | oracle.MODE_C, oracle.MODE_EKC)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("mode", [E, EK, EC, EKC])
def test_supplying_the_absmax_scale_changes_nothing(bits, mode):
    """With s = absmax / qmax handed in, every output equals the default path's bit for bit."""
    for shape in [(6, 9, 3, 3), (4, 33, 1, 1), (3, 5, 5, 5)]:
        w = W.random_layer(shape, seed=bits)
        a = oracle.quantize_layer(w, bits=bits, mode=mode, details=True)
        b = oracle.quantize_layer(w, bits=bits, mode=mode, details=True, scales_in=a.scales)
        for x, y in ((a.codes, b.codes), (a.scales, b.scales), (a.kernel_err, b.kernel_err), (a.channel_err, b.channel_err),
                     (a.pert, b.pert), (a.flip, b.flip)):
            assert np.array_equal(x, y)


def test_hand_worked_clipped_kernel():
    """bits = 4 (codes in [-7, 7]), s = 1, one kernel [9.25, 0.375, 0.375]: 9.25 clips to 7 with
    perturbation -2.25, the others round to 0 with -0.375 each, e = -3.0.  round(3.0) = 3 flips are
    asked for, only the two unclipped elements can move (7 -> 8 leaves the range): both are flipped
    to 1, the kernel keeps e' = -3.0 + 2 = -1.0, and no candidate is left for SQuant-C."""
    w = np.array([[[9.25, 0.375, 0.375]]], dtype=np.float32)
    r = oracle.quantize_layer(w, bits=4, mode=EK, details=True, scales_in=np.array([1.0], np.float32))
    assert r.codes.reshape(-1).tolist() == [7, 1, 1]
    assert r.flip.reshape(-1).tolist() == [0, 1, 1]
    assert r.pert.reshape(-1).tolist() == [-2 ** 31, int(0.625 * ONE), int(0.625 * ONE)]   # the 32-bit view saturates at -2.0
    assert r.kernel_err[0, 0] == -1.0 and r.channel_err[0] == -1.0
    r = oracle.quantize_layer(w, bits=4, mode=EKC, details=True, scales_in=np.array([1.0], np.float32))
    assert r.codes.reshape(-1).tolist() == [7, 1, 1] and r.channel_err[0] == -1.0     # SQuant-C has nothing to flip
    # the mirror image clips at the lower bound (narrow range: -7)
    r = oracle.quantize_layer(-w, bits=4, mode=EK, details=True, scales_in=np.array([1.0], np.float32))
    assert r.codes.reshape(-1).tolist() == [-7, -1, -1] and r.kernel_err[0, 0] == 1.0
    # without the narrow-range flag the lower bound is -8: -9.25 clips to -8, e = +1.25 + 0.75 -> k = 2
    r = oracle.quantize_layer(-w, bits=4, mode=EK, flags=0, details=True, scales_in=np.array([1.0], np.float32))
    assert r.codes.reshape(-1).tolist() == [-8, -1, -1] and r.kernel_err[0, 0] == 0.0


def test_hand_worked_clipped_channel():
    """SQuant-C with a clipped element, a 1x1 layer (every element its own kernel), bits = 4, s = 1:
    [9.0, 0.25, -0.25] rounds to [7, 0, 0] with perturbations [-2, -0.25, +0.25], e_c = -2.0, two
    flips asked for.  Candidates need the sign of e_c and an in-range flip: only the second element
    (the first would go to 8).  It is flipped; the channel keeps -1.0."""
    w = np.array([[9.0, 0.25, -0.25]], dtype=np.float32)
    r = oracle.quantize_layer(w, bits=4, mode=EKC, details=True, scales_in=np.array([1.0], np.float32))
    assert r.codes.reshape(-1).tolist() == [7, 1, 0] and r.flip.reshape(-1).tolist() == [0, 2, 0]
    assert r.channel_err[0] == -1.0 and r.kernel_err.reshape(-1).tolist() == [-2.0, 0.75, 0.25]
    r = oracle.quantize_layer(w, bits=4, mode=EC, details=True, scales_in=np.array([1.0], np.float32))
    assert r.codes.reshape(-1).tolist() == [7, 1, 0] and r.channel_err[0] == -1.0


def test_bad_scales_are_replaced_by_one():
    w = W.random_layer((4, 6, 3, 3), seed=3)
    ref = oracle.quantize_layer(w, bits=4, scales_in=np.ones(4, np.float32))
    for bad in (0.0, -2.0, np.inf, np.nan):
        r = oracle.quantize_layer(w, bits=4, scales_in=np.full(4, bad, np.float32))
        assert np.array_equal(r.scales, np.ones(4, np.float32)) and np.array_equal(r.codes, ref.codes)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("shape", [(12, 7, 3, 3), (9, 40, 1, 1), (5, 6, 2, 2)])
@pytest.mark.parametrize("mode", [EK, EKC, EC])
def test_clipping_invariants(shape, bits, mode):
    """Scales 2 to 4 times too small, so that many elements clip.  Codes stay in range; clipped
    elements are never flipped; an element's perturbation leaves [-0.5, 0.5] only by a flip
    (then 0.5 <= |p| < 1, Eq. 12) or by clipping; every kernel meets |e'| <= 0.5 (Eq. 10) unless it
    ran out of candidates, in which case every in-range element of the sum's sign was flipped; the
    error sums are the sums of the final perturbations."""
    w = W.random_layer(shape, seed=11 * bits)
    qmax = 2 ** (bits - 1) - 1
    m = shape[0]
    sc = (np.abs(w.reshape(m, -1)).max(1) / qmax / np.linspace(2.0, 4.0, m)).astype(np.float32)
    r = oracle.quantize_layer(w, bits=bits, mode=mode, details=True, scales_in=sc)
    e_only = oracle.quantize_layer(w, bits=bits, mode=E, details=True, scales_in=sc)
    x = (w.reshape(m, -1) / sc[:, None]).astype(np.float32)
    clipped = np.abs(np.rint(x)) > qmax
    assert clipped.mean() > 0.05
    codes = r.codes.reshape(m, -1).astype(np.int64)
    assert codes.min() >= -qmax and codes.max() <= qmax
    assert np.array_equal(np.abs(codes[clipped]), np.full(clipped.sum(), qmax))
    assert not r.flip.reshape(m, -1)[clipped].any()
    # pert is exact here (|p| < 2 needs |x| < qmax + 2; check against the definition in float64 where it fits)
    p = codes.astype(np.float64) - x.astype(np.float64)
    fits = np.abs(p) < 1.9
    assert np.array_equal(r.pert.reshape(m, -1)[fits], np.rint(p[fits] * ONE).astype(np.int64).astype(np.int32))
    fl = r.flip.reshape(m, -1)
    flipped = (fl == 1) | (fl == 2)          # 3 = flipped by SQuant-K and flipped back by SQuant-C: as rounded
    assert (np.abs(p[~flipped & ~clipped]) <= 0.5).all() and (np.abs(p[flipped]) >= 0.5).all() and (np.abs(p[flipped]) < 1.0).all()
    # error sums = sums of final perturbations (float64 is exact for these magnitudes)
    k = int(np.prod(shape[2:]))
    ksum = np.rint(p * ONE).reshape(m, shape[1], k).sum(-1)
    assert np.array_equal(r.kernel_err, (ksum / ONE).astype(np.float32))
    assert np.array_equal(r.channel_err, (ksum.sum(1) / ONE).astype(np.float32))
    if mode & oracle.MODE_K:
        # per kernel, from the SQuant-E state: either the bound of Eq. 10 holds, or all candidates went
        pe = np.rint((e_only.codes.reshape(m, -1).astype(np.float64) - x.astype(np.float64)) * ONE).reshape(m, shape[1], k)
        qe = e_only.codes.reshape(m, shape[1], k).astype(np.int64)
        kflip = (r.flip.reshape(m, shape[1], k) & 1) != 0
        ek = oracle.quantize_layer(w, bits=bits, mode=EK, details=True, scales_in=sc)
        ek_sum = np.rint(ek.kernel_err.astype(np.float64) * ONE)
        for c in range(m):
            for n in range(shape[1]):
                e = pe[c, n].sum()
                if e == 0:
                    assert not kflip[c, n].any()
                    continue
                sg = 1 if e > 0 else -1
                cand = (np.sign(pe[c, n]) == sg) & (np.abs(qe[c, n] - sg) <= qmax)
                want = int((abs(e) + HALF - 1) // ONE)
                assert kflip[c, n].sum() == min(want, cand.sum()) and not (kflip[c, n] & ~cand).any()
                if want <= cand.sum():
                    assert abs(ek_sum[c, n]) <= HALF
                else:
                    left = sg * (abs(e) - cand.sum() * ONE)      # reported as fp32: (float)(integer sum) * 2^-30
                    assert ek.kernel_err[c, n] == np.float32(np.float32(left) * np.float32(2.0 ** -30))
    if mode & oracle.MODE_C:
        # SQuant-C: |e_c'| <= 0.5 (Eq. 11) unless the channel ran out of candidates
        cs = np.rint(r.channel_err.astype(np.float64) * ONE)
        ok = np.abs(cs) <= HALF
        cflip = (r.flip.reshape(m, -1) & 2) != 0
        for c in np.nonzero(~ok)[0]:   # every flip went against the sum's sign and one more was not to be had
            assert (np.sign(p[c][cflip[c]]) == -np.sign(cs[c])).all()


@pytest.mark.parametrize("K", [3, 4, 6, 9])
def test_squant_k_with_clipping_is_the_constrained_optimum_bruteforce(K):
    """App. B.2 with the clip of Sec. 2.2: over ALL subsets of one-step flips that keep every code
    in range (any element, either direction), first the distance of |sum| from the allowed 0.5 is
    minimised, then the sum of squared perturbations; the checker's result attains both minima."""
    rng = np.random.default_rng(K)
    bits, qmax = 3, 3
    for trial in range(60):
        x = rng.uniform(-qmax - 2.5, qmax + 2.5, size=K)
        x = np.round(x * 64) / 64                      # exact in fp32, ties and halves included
        w = x.astype(np.float32).reshape(1, 1, K)
        r = oracle.quantize_layer(w, bits=bits, mode=EK, details=True, scales_in=np.array([1.0], np.float32))
        q0 = np.clip(np.rint(x), -qmax, qmax).astype(np.int64)
        got_p = (r.codes.reshape(-1).astype(np.int64) - x) * ONE
        got = (max(abs(got_p.sum()) - HALF, 0), (got_p ** 2).sum())
        best = None
        for moves in itertools.product((-1, 0, 1), repeat=K):
            q = q0 + np.array(moves)
            if np.abs(q).max() > qmax:
                continue
            pp = (q - x) * ONE
            if (np.abs(pp[np.array(moves) != 0]) >= ONE).any():   # a flip moves to the OTHER neighbour of x, not past it
                continue
            key = (max(abs(pp.sum()) - HALF, 0), (pp ** 2).sum())
            if best is None or key < best:
                best = key
        assert got == best, (x.tolist(), r.codes.reshape(-1).tolist(), got, best)
