"""Pins of the oracle's rotary position embedding (CPU only): what the mathematics fixes, none of it a retyping
of the oracle's own formula. A swapped pair, a wrong sign or a transposed table fails at least one."""
import numpy as np

import oracle

F16 = np.float16


def _table(n_pos, hw, base=10000.0):
    """(cos, sin) of angle p * base^(-i/hw), fp32 [n_pos, hw, 2], from fp64."""
    ang = np.arange(n_pos)[:, None] * base ** (-np.arange(hw) / hw)[None, :]
    return np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)


def _rot(x, table, pos):
    return oracle.rope(x, table, pos).view(F16)


def test_matches_a_complex_multiplication_in_fp64_to_half_an_ulp():
    rng = np.random.default_rng(1)
    d, hw, n = 128, 64, 200
    x = rng.standard_normal((n, d)).astype(F16)
    table = _table(512, hw)
    pos = rng.integers(0, 512, n).astype(np.int32)
    got = _rot(x, table, pos).astype(np.float64)
    z = x[:, :hw].astype(np.float64) + 1j * x[:, hw:].astype(np.float64)
    w = z * (table[pos, :, 0].astype(np.float64) + 1j * table[pos, :, 1].astype(np.float64))
    ref = np.concatenate([w.real, w.imag], axis=1)
    ulp = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 2.0 ** -14))) - 10), 2.0 ** -24)
    assert np.all(np.abs(got - ref) <= 0.5 * ulp + 4 * 2.0 ** -24 * np.abs(ref).max())
    # and it is not the identity, the inverse rotation or the interleaved pairing
    wi = z * np.conj(table[pos, :, 0].astype(np.float64) + 1j * table[pos, :, 1].astype(np.float64))
    assert np.abs(got - np.concatenate([wi.real, wi.imag], axis=1)).max() > 0.1
    assert np.abs(got - x.astype(np.float64)).max() > 0.1


def test_position_zero_and_a_zero_angle_are_the_identity_bit_for_bit():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal((50, 64)) * 30).astype(F16)
    table = _table(8, 32)
    assert np.array_equal(oracle.rope(x, table, np.zeros(50, np.int32)), x.view(np.uint16))
    flat = np.zeros((8, 32, 2), np.float32)
    flat[..., 0] = 1.0
    assert np.array_equal(oracle.rope(x, flat, np.arange(50, dtype=np.int32) % 8), x.view(np.uint16))


def test_quarter_turn_swaps_the_halves_with_a_sign():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((10, 128)).astype(F16)
    quarter = np.zeros((1, 64, 2), np.float32)
    quarter[..., 1] = 1.0                                  # cos 0, sin 1
    got = _rot(x, quarter, np.zeros(10, np.int32))
    assert np.array_equal(got[:, :64], -x[:, 64:]) and np.array_equal(got[:, 64:], x[:, :64])


def test_norm_is_preserved_and_inner_products_depend_on_the_distance_only():
    rng = np.random.default_rng(4)
    d, hw = 128, 64
    table = _table(4096, hw)
    q = rng.standard_normal((1, d)).astype(F16)
    k = rng.standard_normal((1, d)).astype(F16)
    dots = []
    for p in (0, 7, 100, 3000):
        qr = _rot(q, table, np.array([p + 17], np.int32)).astype(np.float64)
        kr = _rot(k, table, np.array([p], np.int32)).astype(np.float64)
        assert abs(np.linalg.norm(kr) - np.linalg.norm(k.astype(np.float64))) < 2e-3 * np.linalg.norm(kr)
        dots.append(float((qr * kr).sum()))
    assert max(dots) - min(dots) < 0.05                    # fp16 rounding of 128 terms of size about 1
    other = float((_rot(q, table, np.array([40], np.int32)).astype(np.float64) *
                   _rot(k, table, np.array([0], np.int32)).astype(np.float64)).sum())
    assert abs(other - dots[0]) > 0.05                     # another distance: another value


def test_rounding_is_to_nearest_even_of_the_binary32_sum():
    # x = 1 + 2^-10 (odd last bit), c = 1 + 2^-11 exactly representable in binary32, y = 0: the product is
    # 1 + 2^-10 + 2^-11 + 2^-21, just above a binary16 tie -> rounds up to 1 + 2^-9
    x = np.zeros((1, 2), F16)
    x[0, 0] = F16(1 + 2.0 ** -10)
    t = np.zeros((1, 1, 2), np.float32)
    t[0, 0, 0] = np.float32(1 + 2.0 ** -11)
    got = _rot(x, t, np.zeros(1, np.int32))
    assert got[0, 0] == F16(1 + 2.0 ** -9) and got[0, 1] == 0
    # c = 1 + 2^-11 - 2^-20: the product is 2^-21 (and a little) below the tie -> rounds down
    t[0, 0, 0] = np.float32(1 + 2.0 ** -11 - 2.0 ** -20)
    assert _rot(x, t, np.zeros(1, np.int32))[0, 0] == F16(1 + 2.0 ** -10)
