"""Pins of the oracle's rotary embedding against what the mathematics fixes: complex multiplication, the
relative-position identity, norm preservation, the identity at position 0, a hand-worked pair, and the rounding
bound that ties the execution-datatype variant to the exact one."""

import numpy as np
import pytest

from oracle import apply_rope, rope_frequencies, rotate_exact, round_to_dtype


def _keys(seed, n, d, dtype="bf16"):
    rng = np.random.default_rng(seed)
    return round_to_dtype(rng.standard_normal((3, n, d)), dtype)


def test_frequencies_are_the_geometric_ladder():
    f = rope_frequencies(8, 10000.0)
    assert f[0] == 1.0
    assert np.allclose(f[1:] / f[:-1], 10000.0 ** (-2.0 / 8), rtol=1e-14)
    assert np.isclose(f[-1], 10000.0 ** (-6.0 / 8), rtol=1e-14)


def test_exact_rotation_is_complex_multiplication_on_half_split_pairs():
    d, n = 16, 7
    k = _keys(1, n, d)
    pos = np.array([0, 1, 2, 37, 4095, 32768, 131071])
    z = k[..., : d // 2] + 1j * k[..., d // 2 :]
    w = z * np.exp(1j * np.outer(pos, 10000.0 ** (-2.0 * np.arange(d // 2) / d)))
    r = rotate_exact(k, pos, 10000.0)
    assert np.allclose(r[..., : d // 2], w.real, atol=1e-9)
    assert np.allclose(r[..., d // 2 :], w.imag, atol=1e-9)


def test_hand_worked_pair():
    # d = 2: one pair (x, y) = (1, 0), theta_0 = 1; position p rotates it to (cos p, sin p)
    r = rotate_exact(np.array([[1.0, 0.0]]), [2], 10000.0)
    assert np.allclose(r, [[np.cos(2.0), np.sin(2.0)]], atol=1e-15)
    # d = 4, base 100: theta = (1, 0.1); key (0, 2, 1, 0) at p = 5: pair 0 = (0, 1) -> (-sin 5, cos 5),
    # pair 1 = (2, 0) -> (2 cos 0.5, 2 sin 0.5)
    r = rotate_exact(np.array([[0.0, 2.0, 1.0, 0.0]]), [5], 100.0)
    assert np.allclose(r, [[-np.sin(5.0), 2 * np.cos(0.5), np.cos(5.0), 2 * np.sin(0.5)]], atol=1e-14)


def test_position_zero_is_the_identity_and_norms_are_kept():
    k = _keys(2, 5, 32)
    assert np.array_equal(rotate_exact(k, np.zeros(5), 5e5), k)
    assert np.array_equal(apply_rope(k, np.zeros(5), 5e5, "bf16"), k)
    r = rotate_exact(k, [3, 99, 1000, 65000, 130000], 5e5)
    assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(k, axis=-1), rtol=1e-12)
    h = 16
    assert np.allclose(r[..., :h] ** 2 + r[..., h:] ** 2, k[..., :h] ** 2 + k[..., h:] ** 2, rtol=1e-10, atol=1e-12)


def test_logit_depends_only_on_the_position_difference():
    d = 64
    rng = np.random.default_rng(3)
    q = rng.standard_normal((1, 1, d))
    k = rng.standard_normal((1, 1, d))
    for m, n in [(10, 3), (5000, 4993), (131000, 130993)]:
        a = (rotate_exact(q, [m], 10000.0) * rotate_exact(k, [n], 10000.0)).sum()
        b = (rotate_exact(q, [m - n], 10000.0) * k).sum()
        assert np.isclose(a, b, rtol=1e-9, atol=1e-9)


@pytest.mark.parametrize("dtype,ulp", [("bf16", 2.0 ** -8), ("fp16", 2.0 ** -11)])
def test_execution_datatype_variant_stays_within_its_rounding_bound(dtype, ulp):
    d, n = 128, 64
    k = _keys(4, n, d, dtype)
    pos = 100000 + np.arange(n)
    e = rotate_exact(k, pos, 5e5)
    r = apply_rope(k, pos, 5e5, dtype)
    assert np.array_equal(r, round_to_dtype(r, dtype))  # values of the datatype
    # five roundings (cos, sin, two products, one sum), each at most half an ulp of a term bounded by |x| + |y|
    h = d // 2
    mag = np.abs(k[..., :h]) + np.abs(k[..., h:])
    bound = 3.0 * ulp * np.concatenate([mag, mag], axis=-1) + 1e-30
    assert np.all(np.abs(r - e) <= bound)
    # and a wrong sign or a swapped table would not pass: the error against the inverse rotation is large
    wrong = rotate_exact(k, -pos, 5e5)
    assert np.abs(r - wrong).max() > 0.5


def test_execution_datatype_rotation_bit_for_bit_on_a_hand_worked_pair():
    """d = 2 (one pair, theta = 1), position 1, bf16, every rounding worked by hand (two of them are ties):
    cos 1 = 0.5403023 -> 0.5390625, sin 1 = 0.8414710 -> 0.83984375; (x, y) = (1.5, 2.5):
      x c = 0.80859375 (exact)             y s = 2.099609375 -> 2.09375
      x' = RN(0.80859375 - 2.09375) = RN(-1.28515625), a tie -> -1.28125 (even)
      y c = 1.34765625, a tie -> 1.34375   x s = 1.259765625 -> 1.2578125
      y' = RN(1.34375 + 1.2578125) = RN(2.6015625), a tie -> 2.59375
    Unrounded products would give x' = RN(-1.291015625) = -1.2890625 instead."""
    r = apply_rope(np.array([[1.5, 2.5]]), [1], 10000.0, "bf16")
    assert r.tolist() == [[-1.28125, 2.59375]]
    r0 = apply_rope(np.array([[1.5, 2.5]]), [0], 10000.0, "bf16")
    assert r0.tolist() == [[1.5, 2.5]]
