"""Pins of the decoder-layer operator oracle: closed forms and invariants of the definitions."""
import math

import numpy as np

from oracle.model_ops_oracle import add_rmsnorm, argmax_rows, swiglu


def test_rmsnorm_closed_forms_and_invariants():
    # a constant vector has root mean square |a|: every output is sign(a) (times the weight)
    s, y = add_rmsnorm(np.full(8, -3.0), None, eps=0.0)
    np.testing.assert_allclose(y, -np.ones(8), rtol=1e-15)
    np.testing.assert_array_equal(s, np.full(8, -3.0))
    # (3, 4): mean square 12.5 -> 3 / sqrt(12.5), 4 / sqrt(12.5); weights multiply per coordinate
    _, y = add_rmsnorm([3.0, 4.0], None, weight=[2.0, -1.0], eps=0.0)
    np.testing.assert_allclose(y, [6.0 / math.sqrt(12.5), -4.0 / math.sqrt(12.5)], rtol=1e-15)
    # the output has unit root mean square and does not change when the input is scaled (eps = 0)
    rng = np.random.RandomState(0)
    x = rng.randn(5, 64)
    _, y = add_rmsnorm(x, None, eps=0.0)
    np.testing.assert_allclose(np.sqrt(np.mean(y * y, axis=-1)), np.ones(5), rtol=1e-14)
    np.testing.assert_allclose(add_rmsnorm(7.5 * x, None, eps=0.0)[1], y, rtol=1e-13)
    # eps sits inside the square root, next to the MEAN of the squares (not their sum)
    _, y = add_rmsnorm([1.0, 1.0, 1.0, 1.0], None, eps=3.0)
    np.testing.assert_allclose(y, np.full(4, 0.5), rtol=1e-15)
    # the residual is added before the norm and returned
    s, y = add_rmsnorm([1.0, 2.0], [2.0, 2.0], eps=0.0)
    np.testing.assert_array_equal(s, [3.0, 4.0])
    np.testing.assert_allclose(y, [3.0 / math.sqrt(12.5), 4.0 / math.sqrt(12.5)], rtol=1e-15)


def test_swiglu_closed_forms():
    # silu(0) = 0; silu(x) - silu(-x) = x; silu(x) -> x for large x and -> 0 for very negative x
    np.testing.assert_array_equal(swiglu([0.0, 5.0]), [0.0])
    g = np.array([0.3, 2.0, 7.0])
    one = np.ones(3)
    np.testing.assert_allclose(swiglu(np.concatenate([g, one])) - swiglu(np.concatenate([-g, one])), g, rtol=1e-14)
    np.testing.assert_allclose(swiglu([40.0, 1.0]), [40.0], rtol=1e-15)
    assert abs(swiglu([-40.0, 1.0])[0]) < 1e-15
    # silu(1) = 1 / (1 + e^-1); the second half multiplies
    np.testing.assert_allclose(swiglu([1.0, -3.0]), [-3.0 / (1.0 + math.exp(-1.0))], rtol=1e-15)
    # layout: gate = first half, up = second half of the last dimension
    np.testing.assert_allclose(swiglu([[1.0, 0.0, 2.0, 9.0]]), [[2.0 / (1.0 + math.exp(-1.0)), 0.0]], rtol=1e-15)


def test_argmax_takes_the_lowest_index_of_the_maximum():
    z = np.array([[1.0, 5.0, 5.0, -2.0], [-1.0, -1.0, -7.0, -1.0], [0.0, 0.0, 0.0, 3.0]])
    np.testing.assert_array_equal(argmax_rows(z), [1, 0, 3])
