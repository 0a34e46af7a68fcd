"""Pins for the CPU checker: what the paper and the arithmetic fix, independent of its code.

Each test cites the statement it checks.  Fixed-point unit: 2^-30 (ONE = 2^30, HALF = 2^29).
"""
import itertools

import numpy as np
import pytest

import oracle
from oracle import HALF, ONE
from paper_2202_07471_b200 import workloads as W

E, EK, EC, EKC = (oracle.MODE_E, oracle.MODE_E | oracle.MODE_K, oracle.MODE_E | oracle.MODE_C,
                  oracle.MODE_EKC)

SHAPES = [(8, 16, 3, 3), (5, 7, 1, 1), (4, 3, 7, 7), (16, 1, 3, 3), (3, 33, 2, 2), (2, 300, 1, 1),
          (2, 129, 3, 3), (6, 5, 5, 5)]


def _layer(shape, seed, dist="normal"):
    w = W.random_layer(shape, seed)
    if dist == "coarse":       # values on a coarse grid: many exact ties and exact halves
        w = (np.round(w / np.abs(w).max() * 40) / 8).astype(np.float32)
    return w


def _ksum(pert):
    m, n = pert.shape[:2]
    return pert.reshape(m, n, -1).astype(np.int64).sum(-1)


# ------------------------------------------------------------------ scale and SQuant-E
@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
@pytest.mark.parametrize("shape", SHAPES[:5])
def test_mode_E_is_round_to_nearest(shape, bits):
    """Eq. 9: SQuant-E 'is essentially the rounding method'; scale = absmax / qmax (closed form).
    Cross-checked with numpy's own half-even rint and fp32 division."""
    w = _layer(shape, seed=bits)
    r = oracle.quantize_layer(w, bits=bits, mode=E, details=True)
    qmax = 2 ** (bits - 1) - 1
    m = w.shape[0]
    a = np.abs(w.reshape(m, -1)).max(1)
    s = (a / np.float32(qmax)).astype(np.float32)
    assert np.array_equal(r.scales, s)
    x = w.reshape(m, -1) / s[:, None]
    assert x.dtype == np.float32
    q = np.clip(np.rint(x), -qmax, qmax)
    assert np.array_equal(r.codes.reshape(m, -1), q.astype(np.int8))
    # perturbation = code - scaled weight, |.| <= 0.5 (r_e = 0.5), exact in fixed point
    p = (q.astype(np.float64) - x.astype(np.float64)) * ONE
    assert np.array_equal(r.pert.reshape(m, -1), np.rint(p).astype(np.int32))
    assert np.abs(r.pert).max() <= HALF
    assert not r.flip.any()


def test_half_way_values_round_to_even_and_sign_convention():
    """App. B.1: rounding up gives a positive perturbation (0.7 -> 1 is +0.3)."""
    w = np.array([[127, 0.5, 1.5, 2.5, -0.5, -1.5, 0.7, -0.7]], dtype=np.float32)
    r = oracle.quantize_layer(w, bits=8, mode=E, details=True)
    assert r.codes.reshape(-1).tolist() == [127, 0, 2, 2, 0, -2, 1, -1]
    assert r.pert.reshape(-1)[1:6].tolist() == [-HALF, HALF, -HALF, HALF, -HALF]
    assert r.pert.reshape(-1)[6] > 0 > r.pert.reshape(-1)[7]


# ------------------------------------------------------------------ SQuant-K
@pytest.mark.parametrize("dist", ["normal", "coarse"])
@pytest.mark.parametrize("bits", [3, 4, 8])
@pytest.mark.parametrize("shape", SHAPES)
def test_squant_k_invariants(shape, bits, dist):
    w = _layer(shape, seed=11 * bits, dist=dist)
    re_ = oracle.quantize_layer(w, bits=bits, mode=E, details=True)
    rk = oracle.quantize_layer(w, bits=bits, mode=EK, details=True)
    qmax = 2 ** (bits - 1) - 1
    assert rk.codes.min() >= -qmax and rk.codes.max() <= qmax
    assert np.array_equal(re_.scales, rk.scales)
    flipped = (rk.flip & 1).astype(bool)
    assert not (rk.flip & 2).any()
    # Eq. 12: un-flipped |d| <= 0.5, flipped 0.5 <= |d| < 1.0
    ap = np.abs(rk.pert.astype(np.int64))
    assert ap[~flipped].max(initial=0) <= HALF
    if flipped.any():
        assert ap[flipped].min() >= HALF and ap[flipped].max() < ONE
    # a flip is a +-1 mutation of the rounded code, against the sign of the perturbation
    d = rk.codes.astype(np.int32) - re_.codes.astype(np.int32)
    assert np.array_equal(d != 0, flipped)
    assert np.array_equal(d[flipped], -np.sign(re_.pert[flipped]))
    assert np.array_equal(rk.pert[flipped], re_.pert[flipped] + d[flipped] * ONE)
    assert np.array_equal(rk.pert[~flipped], re_.pert[~flipped])
    # Eq. 10: every kernel |sum| <= 0.5; App. B.1: residual = |k - |e||, flips share e's sign
    e0, e1 = _ksum(re_.pert), _ksum(rk.pert)
    assert np.abs(e1).max() <= HALF
    m, n = e0.shape
    k = flipped.reshape(m, n, -1).sum(-1)
    edge = np.abs(rk.codes).reshape(m, n, -1).max(-1) == qmax   # range exclusion may bind there
    ok = ~edge
    assert np.array_equal(np.abs(e1)[ok], np.abs(k * ONE - np.abs(e0))[ok])
    sgn_el = np.sign(re_.pert).reshape(m, n, -1)
    fl = flipped.reshape(m, n, -1)
    assert np.all((sgn_el == np.sign(e0)[..., None]) | ~fl)
    # App. B.1, second proof: k is the only count that meets the bound; at an exact half the
    # smaller count is taken (target interval (-0.5, 0.5] for e > 0, App. B.3).
    kk = (np.abs(e0) + HALF - 1) >> 30
    assert np.array_equal(k[ok], kk[ok])
    # top-k: inside a kernel no un-flipped same-sign element beats a flipped one
    key = np.where(sgn_el == np.sign(e0)[..., None],
                   np.abs(re_.pert.astype(np.int64)).reshape(m, n, -1), -1)
    lo_flipped = np.where(fl, key, np.iinfo(np.int64).max).min(-1)
    hi_unflipped = np.where(~fl, key, -1).max(-1)
    has = k > 0
    assert np.all(hi_unflipped[has & ok] <= lo_flipped[has & ok])


def _bruteforce_kernel(P):
    """Minimum of sum P'^2 over all flip subsets with |sum P'| <= HALF (exact integers).
    A flip moves an element one step against its rounding direction: P -> P - sign(P) * ONE."""
    P = [int(v) for v in P]
    movable = [i for i, v in enumerate(P) if v != 0]
    best = None
    for r in range(len(movable) + 1):
        for sub in itertools.combinations(movable, r):
            Q = list(P)
            for i in sub:
                Q[i] -= ONE if Q[i] > 0 else -ONE
            if abs(sum(Q)) <= HALF:
                obj = sum(v * v for v in Q)
                if best is None or obj < best:
                    best = obj
    return best


@pytest.mark.parametrize("K", [1, 2, 3, 4, 6, 9])
def test_squant_k_is_the_constrained_optimum_bruteforce(K):
    """App. B.2: under the kernel constraint |sum| <= 0.5 the top-k-perturbation flip set
    minimises the element term; App. B.1 (end): flips of opposite-sign elements never help.
    Brute force over all 2^K flip subsets, any element, on exact integers."""
    n_kernels = 40 if K == 9 else 80
    for dist in ("normal", "coarse"):
        w = _layer((1, n_kernels, K, 1), seed=100 + K, dist=dist)
        w[0, 0, 0, 0] = np.abs(w).max() * 4          # keeps every other code far from the clamp
        re_ = oracle.quantize_layer(w, bits=8, mode=E, details=True)
        rk = oracle.quantize_layer(w, bits=8, mode=EK, details=True)
        for n in range(n_kernels):
            want = _bruteforce_kernel(re_.pert[0, n].reshape(-1))
            got = sum(int(v) ** 2 for v in rk.pert[0, n].reshape(-1))
            assert want is not None and got == want, (dist, n)


# ------------------------------------------------------------------ Algorithm 3 + SQuant-C
def _candidates_from_text(re_, rk):
    """Candidate (value, flat index) per kernel, derived from App. B.3's wording rather than
    from a sorted list: Over SQuant -> among the flipped elements the one with the largest
    post-flip |perturbation| (= smallest before the flip; on ties the last one in flip order,
    i.e. the highest index); Under SQuant -> the un-flipped element, same sign as e, with the
    largest |perturbation| (ties: lowest index)."""
    m, n = re_.pert.shape[:2]
    P0 = re_.pert.reshape(m, n, -1).astype(np.int64)
    P1 = rk.pert.reshape(m, n, -1).astype(np.int64)
    fl = (rk.flip.reshape(m, n, -1) & 1).astype(bool)
    K = P0.shape[-1]
    out = {}
    for mm in range(m):
        for nn in range(n):
            e = int(P0[mm, nn].sum())
            if e == 0:
                continue
            sgn = 1 if e > 0 else -1
            k = int(fl[mm, nn].sum())
            if k * ONE > abs(e):
                best = None
                for i in range(K):
                    if fl[mm, nn, i] and (best is None or abs(P1[mm, nn, i]) >= abs(P1[mm, nn, best])):
                        best = i
            else:
                best = None
                for i in range(K):
                    if (not fl[mm, nn, i]) and np.sign(P0[mm, nn, i]) == sgn:
                        if best is None or abs(P0[mm, nn, i]) > abs(P0[mm, nn, best]):
                            best = i
            if best is not None:
                out[(mm, nn)] = (int(P1[mm, nn, best]), best)
    return out


@pytest.mark.parametrize("dist", ["normal", "coarse"])
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("shape", SHAPES)
def test_squant_c_invariants(shape, bits, dist):
    w = _layer(shape, seed=7 * bits + 1, dist=dist)
    if dist == "coarse" and bits == 4:
        w[:, 0, 0, 0] = np.abs(w).max() * 1.01       # keep the other codes clear of the clamp
    re_ = oracle.quantize_layer(w, bits=bits, mode=E, details=True)
    rk = oracle.quantize_layer(w, bits=bits, mode=EK, details=True)
    rc = oracle.quantize_layer(w, bits=bits, mode=EKC, details=True)
    qmax = 2 ** (bits - 1) - 1
    m, n = w.shape[:2]
    assert rc.codes.min() >= -qmax and rc.codes.max() <= qmax
    byC = (rc.flip & 2).astype(bool)
    assert np.array_equal(rc.flip & 1, rk.flip & 1)
    # Sec. 3.3: SQuant-C flips only one element per kernel
    assert byC.reshape(m, n, -1).sum(-1).max(initial=0) <= 1
    d = rc.codes.astype(np.int32) - rk.codes.astype(np.int32)
    assert np.array_equal(d != 0, byC)
    assert np.array_equal(rc.pert, rk.pert + d * ONE)
    assert np.abs(rc.pert.astype(np.int64)).max() < ONE
    # Eq. 11: channel |sum| <= 0.5; relaxation r_k = 1.0 for the kernels (Sec. 3.3 'Relaxation')
    ek, ec = _ksum(rk.pert), _ksum(rc.pert)
    assert np.abs(ec.sum(1)).max() <= HALF
    assert np.abs(ec).max() <= ONE
    touched = byC.reshape(m, n, -1).any(-1)
    assert np.all(np.abs(ec)[touched] >= HALF)
    # emitted sums are the integer sums scaled by 2^-30
    assert np.array_equal(rc.kernel_err, (ec.astype(np.float32) * np.float32(2.0 ** -30)))
    assert np.array_equal(rc.channel_err, ec.sum(1).astype(np.float32) * np.float32(2.0 ** -30))
    # k_c = round(|e_c|) kernels move, each against the sign of e_c; same tie rule as SQuant-K
    tot = ek.sum(1)
    kc = (np.abs(tot) + HALF - 1) >> 30
    cand = _candidates_from_text(re_, rk)
    for mm in range(m):
        sgn = int(np.sign(tot[mm]))
        pool = {nn: v for (m2, nn), v in cand.items() if m2 == mm and np.sign(v[0]) == sgn
                and abs(int(rk.codes.reshape(m, n, -1)[mm, nn, v[1]]) - sgn) <= qmax}
        want_k = min(int(kc[mm]), len(pool))
        got = np.nonzero(touched[mm])[0].tolist()
        assert len(got) == want_k
        # the moved element of a touched kernel is that kernel's candidate
        for nn in got:
            i = int(np.nonzero(byC.reshape(m, n, -1)[mm, nn])[0][0])
            assert nn in pool and pool[nn][1] == i
            assert d.reshape(m, n, -1)[mm, nn, i] == -sgn
        # top-k over (|v| descending, kernel index ascending)
        order = sorted(pool, key=lambda nn: (-abs(pool[nn][0]), nn))
        assert sorted(order[:want_k]) == got


def test_squant_c_true_channel_sum_not_candidate_sum():
    """Eq. 11 bounds the sum over ALL elements of the channel, so k_c comes from the full sum."""
    w = _layer((4, 64, 3, 3), seed=3)
    rk = oracle.quantize_layer(w, bits=4, mode=EK, details=True)
    rc = oracle.quantize_layer(w, bits=4, mode=EKC, details=True)
    tot = _ksum(rk.pert).sum(1)
    nflip = ((rc.flip & 2) != 0).reshape(4, -1).sum(1)
    assert np.array_equal(nflip, (np.abs(tot) + HALF - 1) >> 30)
    assert nflip.max() >= 1


# ------------------------------------------------------------------ special cases / metamorphic
@pytest.mark.parametrize("bits", [4, 8])
def test_kernel_size_one_skips_squant_k(bits):
    """Sec. 3.4: for FC and 1x1 conv SQuant-K can be skipped - it is a no-op there."""
    w = _layer((6, 200, 1, 1), seed=bits)
    a, b = oracle.quantize_layer(w, bits=bits, mode=E), oracle.quantize_layer(w, bits=bits, mode=EK)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.kernel_err, b.kernel_err)
    c, d = oracle.quantize_layer(w, bits=bits, mode=EC), oracle.quantize_layer(w, bits=bits, mode=EKC)
    assert np.array_equal(c.codes, d.codes) and np.array_equal(c.channel_err, d.channel_err)
    assert not np.array_equal(a.codes, c.codes)


def test_depthwise_channel_step_is_noop():
    """With one kernel per output channel the kernel sum is the channel sum: C has nothing to do."""
    w = _layer((32, 1, 3, 3), seed=9)
    a, b = oracle.quantize_layer(w, mode=EK), oracle.quantize_layer(w, mode=EKC)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.channel_err, b.channel_err)


@pytest.mark.parametrize("mode", [E, EK, EC, EKC])
@pytest.mark.parametrize("shape", SHAPES[:4])
def test_negation_scaling_permutation(shape, mode):
    w = _layer(shape, seed=21)
    r = oracle.quantize_layer(w, mode=mode)
    rn = oracle.quantize_layer(-w, mode=mode)
    assert np.array_equal(rn.codes, -r.codes) and np.array_equal(rn.scales, r.scales)
    assert np.array_equal(rn.kernel_err, -r.kernel_err)
    rs = oracle.quantize_layer(w * np.float32(2.0 ** -7), mode=mode)
    assert np.array_equal(rs.codes, r.codes)
    assert np.array_equal(rs.scales, r.scales * np.float32(2.0 ** -7))
    perm = np.random.default_rng(0).permutation(w.shape[0])
    rp = oracle.quantize_layer(w[perm], mode=mode)
    assert np.array_equal(rp.codes, r.codes[perm]) and np.array_equal(rp.channel_err, r.channel_err[perm])


def test_zero_and_tiny_channels():
    w = _layer((4, 8, 3, 3), seed=2)
    w[1] = 0.0
    w[2] *= np.float32(2.0 ** -110)
    r = oracle.quantize_layer(w)
    assert r.scales[1] == 1.0 and not r.codes[1].any() and r.channel_err[1] == 0.0
    assert r.scales[2] == 1.0 and not r.codes[2].any()
    assert r.codes[0].any() and r.codes[3].any()


def test_single_nonzero_and_constant_channels():
    w = np.zeros((2, 4, 3, 3), dtype=np.float32)
    w[0, 2, 1, 1] = -3.0
    w[1] = 0.25
    r = oracle.quantize_layer(w, bits=4, details=True)
    assert r.codes[0, 2, 1, 1] == -7 and np.count_nonzero(r.codes[0]) == 1
    assert np.all(r.codes[1] == 7) and not r.flip.any()


def test_index_tie_break_is_lowest_flat_index():
    """Equal perturbations: the element (kernel) with the lower flat index is flipped first."""
    w = np.zeros((1, 4, 4), dtype=np.float32)
    w[0, 0, 0] = 127.0
    w[0, 1] = 0.6                                   # four equal +0.4 -> e = 1.6, k = 2
    r = oracle.quantize_layer(w, bits=8, mode=EK, details=True)
    assert r.codes[0, 1].tolist() == [0, 0, 1, 1]
    w = np.zeros((1, 7, 1), dtype=np.float32)
    w[0, 0, 0] = 127.0
    w[0, 1:, 0] = 0.75                              # six kernels +0.25 -> e_c = 1.5 exactly, k_c = 1 (tie -> fewer)
    r = oracle.quantize_layer(w, bits=8, mode=EKC, details=True)
    assert r.codes.reshape(-1).tolist() == [127, 0, 1, 1, 1, 1, 1]
    w = np.zeros((1, 6, 1), dtype=np.float32)
    w[0, 0, 0] = 127.0
    w[0, 1:, 0] = 0.68                              # +0.32 * 5 = 1.6 -> k_c = 2
    r = oracle.quantize_layer(w, bits=8, mode=EKC, details=True)
    assert r.codes.reshape(-1).tolist() == [127, 0, 0, 1, 1, 1]


def test_flip_out_of_range_is_excluded():
    """An element already at the clamp edge is not a flip candidate (codes stay in range)."""
    w = np.array([[[7.0, 7.0, 7.0, 6.6, 6.6, 6.6]]], dtype=np.float32)   # s = 1 with bits = 4
    r = oracle.quantize_layer(w, bits=4, mode=EK, details=True)
    assert r.scales[0] == 1.0
    # rounded: 7 7 7 7 7 7 with +0.4 on the last three -> e = +1.2, k = 1: flip a 6.6 down
    assert r.codes.reshape(-1).tolist() == [7, 7, 7, 6, 7, 7]
    r = oracle.quantize_layer(-w, bits=4, mode=EK, details=True)
    assert r.codes.reshape(-1).tolist() == [-7, -7, -7, -6, -7, -7]
    # wide range allows -8: not needed here, but the range follows the flag
    r = oracle.quantize_layer(-w, bits=4, mode=EK, flags=0, details=True)
    assert r.codes.min() >= -8


def test_stage_nesting():
    """E, E+K, E+K+C differ only by flips: codes differ by at most 1 (K) / 1 more (C back or forth)."""
    w = _layer((8, 32, 3, 3), seed=4)
    a, b, c = (oracle.quantize_layer(w, mode=m_) for m_ in (E, EK, EKC))
    assert np.abs(b.codes.astype(int) - a.codes).max() <= 1
    assert np.abs(c.codes.astype(int) - a.codes).max() <= 1


def test_exactly_integer_kernel_sum_is_under_squant():
    """Algorithm 3: 'Over SQuant' needs k > |e| strictly.  With e = +1.0 exactly, k = 1 = |e| is
    Under SQuant, so the kernel's candidate is the first UN-flipped element (+0.25), not the
    flipped one; SQuant-C may then take it and leave the kernel at -1.0 (r_k = 1.0)."""
    w = np.zeros((1, 6, 4), dtype=np.float32)
    w[0, 0, 0] = 127.0
    w[0, 1] = 0.75                                  # 4 x +0.25 = +1.0 -> k = 1, e' = 0
    w[0, 2:, 0] = 0.8125                            # four kernels at +0.1875 -> e_c = 0.75, k_c = 1
    rk = oracle.quantize_layer(w, bits=8, mode=EK, details=True)
    assert rk.codes[0, 1].tolist() == [0, 1, 1, 1] and rk.kernel_err[0, 1] == 0.0
    rc = oracle.quantize_layer(w, bits=8, mode=EKC, details=True)
    assert rc.codes[0, 1].tolist() == [0, 0, 1, 1]
    assert rc.kernel_err[0].tolist() == [0.0, -1.0, 0.1875, 0.1875, 0.1875, 0.1875]
    assert rc.channel_err[0] == -0.25
    rn = oracle.quantize_layer(-w, bits=8, mode=EKC)
    assert np.array_equal(rn.codes, -rc.codes)


def test_range_exclusion_binds_only_on_a_very_wide_kernel():
    """When absmax / s rounds to just above qmax, that element's perturbation points inward and a
    flip would push its code to qmax + 1.  It has |perturbation| <= one ulp of qmax, so it can
    only be selected when ~2^16 elements tie with it: build exactly that and check the code
    never leaves the range."""
    qmax = np.float32(127.0)
    a = None
    for t in np.linspace(1.0, 2.0, 4000, dtype=np.float32):
        s = np.float32(t) / qmax
        if np.float32(t) / s > qmax:
            a = np.float32(t)
            break
    assert a is not None
    s = a / qmax
    K = 70000
    w = np.full((1, 1, K), s * np.float32(2.0 ** -17), dtype=np.float32)   # each rounds to 0 with -2^-17
    w[0, 0, 0] = a
    r = oracle.quantize_layer(w, bits=8, mode=EK, details=True)
    assert r.scales[0] == s
    assert r.pert[0, 0, 0] == -(1 << 13) and r.pert[0, 0, 1] == ONE - (1 << 13)
    assert r.codes[0, 0, 0] == 127                  # the edge element stayed
    assert r.codes[0, 0, 1] == 1 and int(r.codes[0, 0, 2:].max()) == 0
    assert abs(float(r.kernel_err[0, 0])) <= 0.5


def _unpack_int4(packed, nk):
    u = packed.astype(np.uint8)
    out = np.empty((packed.shape[0], 2 * packed.shape[1]), dtype=np.int16)
    out[:, 0::2] = u & 15
    out[:, 1::2] = u >> 4
    out = np.where(out > 7, out - 16, out)
    return out[:, :nk].astype(np.int8)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("shape", [(5, 7, 3, 3), (4, 33, 1, 1), (3, 2, 5, 5), (2, 1, 3, 3)])
def test_packed_int4_output_is_a_relabelling(shape, bits):
    """Packed output: two's-complement nibbles, low nibble = even flat index, rows of ceil(NK/2)
    bytes; unpacking gives exactly the int8 codes, everything else is unchanged."""
    w = _layer(shape, seed=bits)
    a = oracle.quantize_layer(w, bits=bits, mode=EKC)
    b = oracle.quantize_layer(w, bits=bits, mode=EKC, flags=oracle.FLAG_NARROW_RANGE | oracle.FLAG_PACK_INT4)
    nk = int(np.prod(shape[1:]))
    assert b.codes.shape == (shape[0], (nk + 1) // 2)
    assert np.array_equal(_unpack_int4(b.codes, nk), a.codes.reshape(shape[0], -1))
    assert np.array_equal(a.scales, b.scales) and np.array_equal(a.kernel_err, b.kernel_err)
    if nk & 1:
        assert not ((b.codes[:, -1].astype(np.uint8) >> 4).any())   # pad nibble is zero
    with pytest.raises(ValueError):
        oracle.quantize_layer(w, bits=6, flags=oracle.FLAG_PACK_INT4)


@pytest.mark.parametrize("bits", [4, 8])
def test_dequantized_output_is_code_times_scale(bits):
    """Algorithm 1 returns C * s.  Every quantized weight is within one step of the original
    (Eq. 12: |perturbation| < 1 in units of s), un-flipped ones within half a step."""
    w = _layer((6, 20, 3, 3), seed=bits)
    r = oracle.quantize_layer(w, bits=bits, mode=EKC, details=True)
    s = r.scales[:, None, None, None]
    assert np.array_equal(r.dequant, r.codes.astype(np.float32) * s)
    err = np.abs(r.dequant.astype(np.float64) - w) / s
    assert err.max() < 1.0 + 1e-6
    assert err[r.flip == 0].max() <= 0.5 + 1e-6


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_dequantized_bf16_output_matches_the_library_conversion(bits):
    """Algorithm 1 returns C * s; as bfloat16 it is the fp32 product rounded to nearest even.
    Cross-checked with PyTorch's own fp32 -> bfloat16 conversion (an independent routine)."""
    import torch
    w = _layer((6, 40, 3, 3), seed=30 + bits)
    w[2] *= np.float32(2.0 ** 40)
    w[3] *= np.float32(2.0 ** -40)
    r = oracle.quantize_layer(w, bits=bits, details=True)
    want = torch.from_numpy(r.dequant).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(r.dequant_bf16, want)
    assert (r.dequant_bf16 != (r.dequant.view(np.uint32) >> 16).astype(np.uint16)).any()   # rounding, not truncation, is exercised
