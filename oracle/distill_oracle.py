"""Plain fp64 CPU oracle for the distillation loss of Breadcrumbs Reasoning (Section 3.2, Eq. 1).

TEST INFRASTRUCTURE: only tests/, the smoke entry and the benchmark's CPU-baseline leg may import
this module; the product path never does.  It shares no code with the CUDA kernels.

Eq. 1: for a trajectory x sampled from the teacher, L(x) = (1/|x|) sum_i KL(teacher(. | x_<i) ||
student(. | x_<i)), and the batch loss is the mean of L(x_b) over the B trajectories (a mean of
per-trajectory means, not a mean over all tokens).  Only the student receives gradients.

The teacher distributions are stored as the top-K entries per position (Implementation Details:
the top 100 logits per time step, which cover more than 90 % of the probability mass).  Reading
taken here (the paper does not say how the stored entries are normalised): the stored values are
the teacher's log-probabilities under its full-vocabulary normalisation, and the KL sum runs over
the stored entries only,
    KL_K(p || q) = sum_{k in top-K} p_k (log p_k - log q_k),
with q the student's softmax over the whole vocabulary.  With K = |V| this is Eq. 1 exactly.
"""
from __future__ import annotations

import numpy as np

__all__ = ["log_softmax", "row_losses", "batch_loss", "loss_gradient"]


def log_softmax(z):
    """Row-wise log-softmax of logits z [rows, V], fp64."""
    z = np.asarray(z, dtype=np.float64)
    m = z.max(axis=1, keepdims=True)
    return z - m - np.log(np.exp(z - m).sum(axis=1, keepdims=True))


def row_losses(student_logits, teacher_idx, teacher_logprob):
    """KL_K per position: student_logits [rows, V]; teacher_idx [rows, K] (int); teacher_logprob
    [rows, K].  Entries with teacher_logprob = -inf carry no mass and contribute nothing."""
    lq = log_softmax(student_logits)
    idx = np.asarray(teacher_idx, dtype=np.int64)
    lp = np.asarray(teacher_logprob, dtype=np.float64)
    out = np.zeros(lq.shape[0])
    for r in range(lq.shape[0]):
        for k in range(idx.shape[1]):
            if np.isfinite(lp[r, k]):
                out[r] += np.exp(lp[r, k]) * (lp[r, k] - lq[r, idx[r, k]])
    return out


def batch_loss(row_loss, cu_rows):
    """Eq. 1: mean over trajectories of the mean over each trajectory's positions.  cu_rows: prefix
    sums [B + 1] of the trajectories' lengths; empty trajectories contribute zero."""
    row_loss = np.asarray(row_loss, dtype=np.float64)
    B = len(cu_rows) - 1
    total = 0.0
    for b in range(B):
        a, e = cu_rows[b], cu_rows[b + 1]
        if e > a:
            total += row_loss[a:e].sum() / (e - a)
    return total / B


def loss_gradient(student_logits, teacher_idx, teacher_logprob, cu_rows):
    """d batch_loss / d student_logits [rows, V]: for a position r of trajectory b,
    w_r * (q_j * sum_k p_k - p_j [j stored]) with w_r = 1 / (B * |x_b|)."""
    lq = log_softmax(student_logits)
    q = np.exp(lq)
    idx = np.asarray(teacher_idx, dtype=np.int64)
    lp = np.asarray(teacher_logprob, dtype=np.float64)
    B = len(cu_rows) - 1
    g = np.zeros_like(q)
    for b in range(B):
        a, e = cu_rows[b], cu_rows[b + 1]
        for r in range(a, e):
            w = 1.0 / (B * (e - a))
            p = np.where(np.isfinite(lp[r]), np.exp(lp[r]), 0.0)
            g[r] = w * p.sum() * q[r]
            for k in range(idx.shape[1]):
                g[r, idx[r, k]] -= w * p[k]
    return g
