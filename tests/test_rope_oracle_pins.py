"""Pins of the rotary-embedding oracle: what the definition fixes, not a retyped formula."""
import math

import numpy as np

from oracle.rope_oracle import rope, split_and_rope


def test_position_zero_is_identity_and_norms_are_kept():
    rng = np.random.RandomState(0)
    x = rng.randn(5, 3, 16)
    np.testing.assert_array_equal(rope(x, 0), x)
    y = rope(x, 37, theta=1e6)
    half = 8
    np.testing.assert_allclose(y[..., :half] ** 2 + y[..., half:] ** 2, x[..., :half] ** 2 + x[..., half:] ** 2, rtol=1e-12)
    assert not np.allclose(y, x)


def test_worked_example_by_hand():
    """D = 4, theta = 10000, pos = 2: pair 0 = (x0, x2) turns by 2 rad, pair 1 = (x1, x3) by 2 / 100 rad."""
    x = np.array([1.0, 2.0, 3.0, 4.0])
    a0, a1 = 2.0, 0.02
    want = np.array([1 * math.cos(a0) - 3 * math.sin(a0), 2 * math.cos(a1) - 4 * math.sin(a1),
                     3 * math.cos(a0) + 1 * math.sin(a0), 4 * math.cos(a1) + 2 * math.sin(a1)])
    np.testing.assert_allclose(rope(x, 2, theta=10000.0), want, rtol=0, atol=1e-14)
    # a quarter turn of a unit vector on the first pair: (1, 0) -> (0, 1); a wrong sign of the sine gives (0, -1)
    e = np.array([1.0, 0.0])
    np.testing.assert_allclose(rope(e, math.pi / 2, theta=7.0), [0.0, 1.0], atol=1e-15)


def test_rotations_add_up_and_scores_depend_on_the_distance_only():
    rng = np.random.RandomState(1)
    q, k = rng.randn(32), rng.randn(32)
    np.testing.assert_allclose(rope(rope(q, 5), 9), rope(q, 14), atol=1e-12)
    s = [rope(q, m) @ rope(k, n) for m, n in ((10, 3), (107, 100), (7, 0))]
    np.testing.assert_allclose(s, [s[0]] * 3, atol=1e-11)
    assert abs(rope(q, 10) @ rope(k, 4) - s[0]) > 1e-3          # another distance, another score


def test_split_layout():
    """Packed rows are [q heads | k heads | v heads]; q and k are rotated with the row's own position, v is not."""
    Hq, Hkv, D = 4, 2, 8
    qkv = np.arange(3 * (Hq + 2 * Hkv) * D, dtype=np.float64).reshape(3, -1)
    q, k, v = split_and_rope(qkv, [0, 1, 5], Hq, Hkv, D)
    np.testing.assert_array_equal(q[0].ravel(), qkv[0, :Hq * D])                     # position 0: untouched
    np.testing.assert_array_equal(v[2].ravel(), qkv[2, (Hq + Hkv) * D:])
    np.testing.assert_allclose(k[2, 1], rope(qkv[2, (Hq + 1) * D:(Hq + 2) * D], 5), atol=1e-12)
    np.testing.assert_allclose(q[1, 3], rope(qkv[1, 3 * D:4 * D], 1), atol=1e-12)
