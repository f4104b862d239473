"""Pins for the oracle's subspace construction (mean and CGS2).

Every check compares the oracle with something other than itself: closed
forms on integer inputs, numpy's Householder QR, brute-force least squares,
and the invariants an orthonormal basis of span{w_i} must satisfy.
"""

import os

import numpy as np
import pytest
import torch

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _traj(D, n, step=0.01, drift=0.002, seed=0):
    W = inputs.trajectory_candidates(D, n, step, drift, seed, "cpu")
    return W[:, :D].numpy().T        # (D, n) view, contiguous columns


# ------------------------------------------------------------------ mean
def test_mean_closed_form_integers():
    # columns 1..n times a fixed integer vector: mean is (n+1)/2 times it
    base = np.array([3, -1, 4, 1, -5, 9, 2, -6], dtype=np.float32)
    n = 7
    W = np.stack([(i + 1) * base for i in range(n)], axis=1)
    np.testing.assert_array_equal(orc.mean(W), (n + 1) / 2.0 * base.astype(np.float64))


def test_mean_is_not_a_sum_or_a_column():
    W = np.array([[1, 2, 6], [0, 0, 3]], dtype=np.float32)
    np.testing.assert_allclose(orc.mean(W), [3.0, 1.0], rtol=0, atol=0)


# ------------------------------------------------------------------ CGS2
def test_cgs2_orthonormal_to_1e12_on_correlated_trajectory():
    A = _traj(20000, 12)
    Q, R, bad = orc.cgs2(A)
    assert bad is None
    G = Q.T @ Q
    assert np.max(np.abs(G - np.eye(12))) <= 1e-12


def test_cgs2_factorisation_is_the_unique_positive_qr():
    A = _traj(5000, 8, seed=3)
    Q, R, bad = orc.cgs2(A)
    assert bad is None
    A64 = A.astype(np.float64)
    # Q^T A is upper triangular with positive diagonal, and Q (Q^T A) = A
    T = Q.T @ A64
    assert np.max(np.abs(np.tril(T, -1))) <= 1e-12 * np.max(np.abs(T))
    assert np.all(np.diag(T) > 0)
    assert np.linalg.norm(A64 - Q @ T) / np.linalg.norm(A64) <= 1e-12
    np.testing.assert_allclose(R, np.triu(T), rtol=0, atol=1e-11 * np.max(np.abs(T)))
    # library Householder QR after fixing the signs of its diagonal
    Qh, Rh = np.linalg.qr(A64)
    sgn = np.sign(np.diag(Rh))
    Qh = Qh * sgn
    Rh = (Rh.T * sgn).T
    kappa = np.linalg.cond(A64)
    assert np.max(np.abs(Q - Qh)) <= 50 * kappa * np.finfo(np.float64).eps
    np.testing.assert_allclose(R, Rh, rtol=0, atol=1e-11 * np.max(np.abs(Rh)))


def test_cgs2_column_order_matters_first_column_is_w0_direction():
    A = _traj(3000, 5, seed=1)
    Q, _, _ = orc.cgs2(A)
    a0 = A[:, 0].astype(np.float64)
    np.testing.assert_allclose(Q[:, 0], a0 / np.linalg.norm(a0), rtol=0, atol=1e-15)


def test_cgs2_n1_and_already_orthonormal_input():
    rng = np.random.default_rng(0)
    v = rng.standard_normal((257, 1)).astype(np.float32)
    Q, R, bad = orc.cgs2(v)
    assert bad is None
    np.testing.assert_allclose(Q[:, 0], v[:, 0].astype(np.float64) / np.linalg.norm(v.astype(np.float64)),
                               atol=1e-15)
    # signed permutation columns are exactly orthonormal in float32: returned unchanged
    E = np.zeros((9, 4), dtype=np.float32)
    E[2, 0] = 1
    E[7, 1] = 1
    E[0, 2] = 1
    E[5, 3] = 1
    Q, R, bad = orc.cgs2(E)
    assert bad is None
    np.testing.assert_array_equal(Q, E.astype(np.float64))
    np.testing.assert_array_equal(R, np.eye(4))


def test_cgs2_positive_diagonal_even_for_negated_columns():
    A = _traj(2000, 4, seed=5).copy()
    A[:, 2] *= -1
    Q, R, _ = orc.cgs2(A)
    assert np.all(np.diag(R) > 0)
    assert np.linalg.norm(A.astype(np.float64) - Q @ R) / np.linalg.norm(A) <= 1e-12


def test_cgs2_duplicate_column_is_rank_deficient():
    A = _traj(1000, 5, seed=2).copy()
    A[:, 3] = A[:, 1]
    _, _, bad = orc.cgs2(A)
    assert bad == 3
    B = _traj(1000, 5, seed=2).copy()
    B[:, 4] = -2 * B[:, 0]                       # exact in float32
    assert orc.cgs2(B)[2] == 4
    C = _traj(1000, 5, seed=2).copy()
    C[:, 4] = 2 * C[:, 0] - C[:, 2]              # dependent up to float32 rounding
    assert orc.cgs2(C)[2] is None
    assert orc.cgs2(C, rel_tol=1e-5)[2] == 4


def test_second_pass_is_needed_single_pass_fails_the_pin():
    """The re-orthogonalisation is what buys 1e-12: a one-pass classical
    Gram-Schmidt written here fails the same check on the same input."""
    A = _traj(20000, 12, step=0.0005, drift=0.0).astype(np.float64)
    n = A.shape[1]
    Q1 = np.zeros_like(A)
    for j in range(n):
        v = A[:, j] - Q1[:, :j] @ (Q1[:, :j].T @ A[:, j])
        Q1[:, j] = v / np.linalg.norm(v)
    assert np.max(np.abs(Q1.T @ Q1 - np.eye(n))) > 1e-12
    Q, _, bad = orc.cgs2(A.astype(np.float32))
    assert bad is None
    assert np.max(np.abs(Q.T @ Q - np.eye(n))) <= 1e-12


def test_orthogonalisation_gives_zero_correlation_where_raw_candidates_have_099():
    raw_cos, orth_cos, _ = [float(x) for x in
                            [l for l in open(os.path.join(GOLDEN, "paper_decoupling.txt"))
                             if not l.startswith("#")][0].split()]
    A = _traj(50000, 10, step=0.003, drift=0.001)
    A64 = A.astype(np.float64)
    An = A64 / np.linalg.norm(A64, axis=0)
    C = An.T @ An
    off = C[~np.eye(10, dtype=bool)]
    assert off.mean() >= raw_cos - 0.02          # candidates: about 0.99, as in the paper
    Q, _, _ = orc.cgs2(A)
    Cq = Q.T @ Q
    assert np.max(np.abs(Cq[~np.eye(10, dtype=bool)])) <= 1e-12   # paper prints 0
    assert orth_cos == 0


# ------------------------------------------------------------------ span
def test_span_properties():
    D, n = 4000, 7
    A = _traj(D, n, seed=4)
    A64 = A.astype(np.float64)
    Q, _, _ = orc.cgs2(A)
    # every candidate is recovered: Q Q^T w_i = w_i
    for i in range(n):
        rec = Q @ (Q.T @ A64[:, i])
        assert np.linalg.norm(rec - A64[:, i]) <= 1e-12 * np.linalg.norm(A64[:, i])
    # and w_bar + Q Q^T (w_i - w_bar) = w_i  (w_bar lies in the span)
    wbar = orc.mean(A)
    for i in range(n):
        rec = wbar + Q @ (Q.T @ (A64[:, i] - wbar))
        assert np.linalg.norm(rec - A64[:, i]) <= 1e-12 * np.linalg.norm(A64[:, i])
    # a vector made orthogonal to all candidates (by a library least-squares solve) projects to 0
    rng = np.random.default_rng(7)
    x = rng.standard_normal(D)
    coef, *_ = np.linalg.lstsq(A64, x, rcond=None)
    x_perp = x - A64 @ coef
    assert np.max(np.abs(Q.T @ x_perp)) <= 1e-10 * np.linalg.norm(x)
    # Q^T x are the least-squares coefficients of x in the basis Q
    c_ls, *_ = np.linalg.lstsq(Q, x, rcond=None)
    np.testing.assert_allclose(Q.T @ x, c_ls, rtol=0, atol=1e-12 * np.linalg.norm(x))
    # Q Q^T x equals the normal-equations projector A (A^T A)^-1 A^T x
    proj_ne = A64 @ np.linalg.solve(A64.T @ A64, A64.T @ x)
    assert np.linalg.norm(Q @ (Q.T @ x) - proj_ne) <= 1e-8 * np.linalg.norm(x)


def test_multi_trajectory_candidates_full_rank():
    W = inputs.multi_trajectory_candidates(6000, 3, 4, 0.005, 0.001, 0, "cpu")
    A = W[:, :6000].numpy().T
    Q, _, bad = orc.cgs2(A)
    assert bad is None
    assert np.max(np.abs(Q.T @ Q - np.eye(12))) <= 1e-12
