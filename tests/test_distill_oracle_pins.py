"""Pins of the distillation-loss oracle (Eq. 1) to facts fixed by the mathematics and to library
routines it does not call itself."""
import math

import numpy as np
import pytest
from scipy.special import log_softmax as sp_log_softmax, rel_entr

from oracle.distill_oracle import batch_loss, log_softmax, loss_gradient, row_losses


def _full(rng, rows, V):
    """Teacher given on the whole vocabulary (K = V): Eq. 1 without truncation."""
    zt = rng.standard_normal((rows, V)) * 2
    lp = sp_log_softmax(zt, axis=1)
    idx = np.tile(np.arange(V), (rows, 1))
    return idx, lp


def test_equal_distributions_give_zero():
    rng = np.random.RandomState(0)
    z = rng.standard_normal((5, 37))
    idx = np.tile(np.arange(37), (5, 1))
    assert np.abs(row_losses(z, idx, sp_log_softmax(z, axis=1))).max() < 1e-12
    assert np.abs(row_losses(z + 3.7, idx, sp_log_softmax(z, axis=1))).max() < 1e-12   # shift invariance of the student


def test_two_class_closed_form():
    # teacher (0.8, 0.2), student logits (0, ln 3) -> q = (0.25, 0.75)
    z = np.array([[0.0, math.log(3.0)]])
    lp = np.log(np.array([[0.8, 0.2]]))
    want = 0.8 * math.log(0.8 / 0.25) + 0.2 * math.log(0.2 / 0.75)
    assert row_losses(z, np.array([[0, 1]]), lp)[0] == pytest.approx(want, abs=1e-14)
    # swapped storage order of the teacher entries: same value
    assert row_losses(z, np.array([[1, 0]]), lp[:, ::-1])[0] == pytest.approx(want, abs=1e-14)


def test_one_hot_teacher_against_uniform_student_is_log_vocab():
    V = 1000
    z = np.full((1, V), 0.3)
    lp = np.array([[0.0, -np.inf]])
    assert row_losses(z, np.array([[17, 4]]), lp)[0] == pytest.approx(math.log(V), abs=1e-12)


def test_full_vocabulary_equals_library_relative_entropy():
    rng = np.random.RandomState(1)
    z = rng.standard_normal((6, 50)) * 3
    idx, lp = _full(rng, 6, 50)
    want = rel_entr(np.exp(lp), np.exp(sp_log_softmax(z, axis=1))).sum(axis=1)
    assert np.allclose(row_losses(z, idx, lp), want, rtol=0, atol=1e-12)
    assert np.allclose(log_softmax(z), sp_log_softmax(z, axis=1), atol=1e-13)


def test_truncated_sum_keeps_only_stored_entries():
    rng = np.random.RandomState(2)
    V, K = 40, 7
    z = rng.standard_normal((3, V))
    idx_full, lp_full = _full(rng, 3, V)
    top = np.argsort(-lp_full, axis=1)[:, :K]
    lp_top = np.take_along_axis(lp_full, top, axis=1)
    lq = sp_log_softmax(z, axis=1)
    want = (np.exp(lp_top) * (lp_top - np.take_along_axis(lq, top, axis=1))).sum(axis=1)
    assert np.allclose(row_losses(z, top, lp_top), want, atol=1e-13)
    # the stored mass is below one, so the truncated value is not the full divergence
    assert np.exp(lp_top).sum(axis=1).max() < 1.0
    assert not np.allclose(row_losses(z, top, lp_top), row_losses(z, idx_full, lp_full))


def test_batch_loss_is_a_mean_of_trajectory_means():
    rows = np.array([1.0, 3.0, 10.0])                 # trajectory 0: two positions, trajectory 1: one
    assert batch_loss(rows, [0, 2, 3]) == pytest.approx(0.5 * (2.0 + 10.0))
    assert batch_loss(rows, [0, 2, 3]) != pytest.approx(rows.mean())
    assert batch_loss(rows, [0, 3, 3]) == pytest.approx(0.5 * (14.0 / 3.0))        # an empty trajectory adds zero


def test_gradient_matches_finite_differences():
    rng = np.random.RandomState(3)
    V, K = 12, 5
    z = rng.standard_normal((4, V))
    idx_full, lp_full = _full(rng, 4, V)
    top = np.argsort(-lp_full, axis=1)[:, :K]
    lp_top = np.take_along_axis(lp_full, top, axis=1)
    cu = [0, 3, 4]
    g = loss_gradient(z, top, lp_top, cu)
    f = lambda zz: batch_loss(row_losses(zz, top, lp_top), cu)
    eps = 1e-6
    for r, j in [(0, 0), (1, 5), (2, 11), (3, 3), (3, int(top[3, 0]))]:
        zp, zm = z.copy(), z.copy()
        zp[r, j] += eps; zm[r, j] -= eps
        assert g[r, j] == pytest.approx((f(zp) - f(zm)) / (2 * eps), abs=1e-8)
    # with the whole vocabulary stored the gradient is w (q - p) and sums to zero over the vocabulary
    gf = loss_gradient(z, idx_full, lp_full, cu)
    w = np.array([1 / 6, 1 / 6, 1 / 6, 1 / 2])[:, None]
    assert np.allclose(gf, w * (np.exp(sp_log_softmax(z, axis=1)) - np.exp(lp_full)), atol=1e-13)
    assert np.abs(gf.sum(axis=1)).max() < 1e-13
