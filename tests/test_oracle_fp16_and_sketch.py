"""Pins for the oracle's binary16 conversions and Eq. 2 / Eq. 3 (CPU only).

Each check compares the oracle with something other than itself: numpy's own
float16 type, a numpy matmul, the closed form of Prop. 1, or values worked by
hand.
"""
import math

import numpy as np
import pytest

import oracle


# ---------------------------------------------------------------- binary16 --
def test_half_to_double_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.half_to_double(int(b)) for b in bits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    # sign of zero survives
    assert math.copysign(1.0, oracle.half_to_double(0x8000)) == -1.0


def _np_half_bits(x):
    with np.errstate(over="ignore"):
        return int(np.array([x], dtype=np.float64).astype(np.float16).view(np.uint16)[0])


def test_double_to_half_rne_matches_numpy_random_and_midpoints():
    rng = np.random.default_rng(1)
    xs = list(rng.standard_normal(20000) * np.exp(rng.uniform(-20, 12, 20000)))
    # exact midpoints between neighbouring halves (ties-to-even), normal and subnormal
    for b in list(range(0, 0x7bff, 37)) + [0, 1, 2, 0x3ff, 0x400, 0x401, 0x7bfe]:
        lo = float(np.array([b], dtype=np.uint16).view(np.float16)[0])
        hi = float(np.array([b + 1], dtype=np.uint16).view(np.float16)[0])
        mid = (lo + hi) / 2.0
        xs += [mid, np.nextafter(mid, 0.0), np.nextafter(mid, np.inf), -mid]
    xs += [65504.0, 65519.999, 65520.0, 65536.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25,
           np.nextafter(2.0 ** -25, 1.0), 2.0 ** -26, 0.0]
    for x in xs:
        assert oracle.double_to_half_rne(float(x)) == _np_half_bits(float(x)), x
    assert oracle.double_to_half_rne(-0.0) == 0x8000


# ---------------------------------------------------------------- Eq. 2 ----
def test_sketch_hand_worked_orientation_and_sign_of_zero():
    # d = 3, m = 4. Rt[i][j]: column j is the j-th hyperplane (row j of the paper's R).
    Rt = np.array([[1.0, 0.0, -1.0, 2.0],
                   [0.0, 1.0, 1.0, -1.0],
                   [2.0, -3.0, 0.0, 0.0]], dtype=np.float32)
    k = np.array([[1.0, 2.0, -1.0]], dtype=np.float16)
    # y0 = 1*1 + 2*0 + (-1)*2 = -1 ; y1 = 0 + 2 + 3 = 5 ; y2 = -1 + 2 + 0 = 1 ; y3 = 2 - 2 + 0 = 0
    bits, y, a = oracle.sketch(k, Rt, want_margin=True)
    assert y.tolist() == [[-1.0, 5.0, 1.0, 0.0]]
    assert bits.tolist() == [[0, 1, 1, 1]]          # sign(0) = +1
    assert a.tolist() == [[3.0, 5.0, 3.0, 4.0]]
    # an all-zero vector gives all ones
    z = oracle.sketch(np.zeros((1, 3), dtype=np.float16), Rt)
    assert z.tolist() == [[1, 1, 1, 1]]


def test_sketch_matches_numpy_matmul_signs_away_from_zero():
    rng = np.random.default_rng(2)
    d, m, rows = 128, 256, 64
    Rt = rng.standard_normal((d, m)).astype(np.float32)
    x = rng.standard_normal((rows, d)).astype(np.float16)
    bits, y, a = oracle.sketch(x, Rt, want_margin=True)
    y_np = x.astype(np.float64) @ Rt.astype(np.float64)
    assert np.allclose(y, y_np, rtol=0, atol=1e-10)
    far = np.abs(y_np) > 1e-9 * a
    assert np.array_equal(bits[far], (y_np[far] >= 0).astype(np.uint8))
    assert np.allclose(a, np.abs(x.astype(np.float64))[:, :, None].__mul__(np.abs(Rt.astype(np.float64))[None]).sum(1))


def test_sketch_scale_invariance_and_negation():
    rng = np.random.default_rng(3)
    d, m = 64, 128
    Rt = rng.standard_normal((d, m)).astype(np.float32)
    x = rng.standard_normal((8, d)).astype(np.float16)
    b1 = oracle.sketch(x, Rt)
    assert np.array_equal(b1, oracle.sketch((x * np.float16(4.0)).astype(np.float16), Rt))
    assert np.array_equal(b1, oracle.sketch((x * np.float16(0.25)).astype(np.float16), Rt))
    bneg, y, _ = oracle.sketch((-x).astype(np.float16), Rt, want_margin=True)
    nz = y != 0
    assert np.array_equal(bneg[nz], 1 - b1[nz])


@pytest.mark.parametrize("theta", [0.0, math.pi / 6, 1.0, math.pi / 2, 2.5, math.pi])
def test_bit_agreement_rate_tracks_one_minus_theta_over_pi(theta):
    """Prop. 1 / Eq. 1: P[bits agree] = 1 - theta/pi for Gaussian hyperplanes."""
    rng = np.random.default_rng(int(theta * 1000) + 11)
    d, m = 16, 1 << 17
    Rt = rng.standard_normal((d, m)).astype(np.float32)
    # a random orthonormal pair (u, w); q = u, k = cos(theta) u + sin(theta) w, rounded to fp16
    Q, _ = np.linalg.qr(rng.standard_normal((d, 2)))
    q = Q[:, 0].astype(np.float16)
    k = (math.cos(theta) * Q[:, 0] + math.sin(theta) * Q[:, 1]).astype(np.float16)
    if theta == 0.0:
        k = q.copy()
    if theta == math.pi:
        k = (-q).astype(np.float16)
    qd, kd = q.astype(np.float64), k.astype(np.float64)
    cosang = float(qd @ kd / (np.linalg.norm(qd) * np.linalg.norm(kd)))
    th = math.acos(max(-1.0, min(1.0, cosang)))      # the angle of the vectors actually used
    bits = oracle.sketch(np.stack([q, k]), Rt)
    agree = float((bits[0] == bits[1]).mean())
    p = 1.0 - th / math.pi
    sigma = math.sqrt(max(p * (1 - p), 1e-12) / m)
    if theta in (0.0, math.pi):
        assert agree == p                          # exact: all agree / all differ
    else:
        assert abs(agree - p) < 4 * sigma + 1e-9, (agree, p, sigma)
    # Eq. 3 on the same bits: alpha = 1 - 2 * (fraction disagreeing)
    sc = oracle.scores(bits[0], bits[1:2])
    assert sc[0] == m - 2 * int((bits[0] != bits[1]).sum())
    assert abs(sc[0] / m - (1 - 2 * th / math.pi)) < 8 * sigma + 1e-9


# ---------------------------------------------------------------- Eq. 3 ----
def test_scores_equal_pm1_inner_product_numpy():
    rng = np.random.default_rng(5)
    for m in (32, 64, 128, 256, 512):
        qb = rng.integers(0, 2, m, dtype=np.uint8)
        kb = rng.integers(0, 2, (100, m), dtype=np.uint8)
        sc = oracle.scores(qb, kb)
        pm = (2 * kb.astype(np.int64) - 1) @ (2 * qb.astype(np.int64) - 1)
        assert np.array_equal(sc, pm)
        ham = (kb != qb[None]).sum(1)
        assert np.array_equal(sc, m - 2 * ham)
    # extremes: identical sketch -> m, complement -> -m
    assert oracle.scores(qb, qb[None])[0] == m
    assert oracle.scores(qb, (1 - qb)[None])[0] == -m


def test_scores_hand_worked():
    q = np.array([1, 0, 1, 1], dtype=np.uint8)
    k = np.array([[1, 0, 1, 1], [0, 0, 1, 1], [0, 1, 0, 0], [1, 1, 0, 1]], dtype=np.uint8)
    assert oracle.scores(q, k).tolist() == [4, 2, -4, 0]
