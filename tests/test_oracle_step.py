"""Pins for the oracle's projection, coefficient update, lift and whole step."""

import numpy as np

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import inputs


def _quantised_basis(D, n, bits, seed=0):
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, seed, "cpu")
    A = W[:, :D].numpy().T
    Q, _, _ = orc.cgs2(A)
    P32 = np.asfortranarray(Q.astype(np.float32))
    codes, s = orc.quantize(P32, bits)
    return A, P32, codes, s


def test_project_and_lift_equal_dense_gemv():
    D, n = 777, 6
    rng = np.random.default_rng(0)
    for bits in (8, 4):
        _, _, codes, s = _quantised_basis(D, n, bits)
        Pt = codes.astype(np.float64) * s.astype(np.float64)[None, :]      # dense P~
        g = (rng.standard_normal(D) * 1e-3).astype(np.float32)
        alpha = rng.standard_normal(n)
        base = rng.standard_normal(D).astype(np.float32)
        np.testing.assert_allclose(orc.project(codes, s, g), Pt.T @ g.astype(np.float64),
                                   rtol=1e-13, atol=1e-18)
        np.testing.assert_allclose(orc.lift(codes, s, alpha, base),
                                   base.astype(np.float64) + Pt @ alpha, rtol=1e-13, atol=1e-16)
        np.testing.assert_allclose(orc.lift(codes, s, alpha, None), Pt @ alpha,
                                   rtol=1e-13, atol=1e-16)


def test_project_and_lift_brute_force_loops():
    codes = np.array([[1, -2], [3, 4], [-5, 6]], dtype=np.int8)
    s = np.array([0.5, 0.25], dtype=np.float32)
    g = np.array([2.0, -1.0, 4.0], dtype=np.float32)
    # c_0 = 0.5*(1*2 + 3*-1 + -5*4) = -10.5 ; c_1 = 0.25*(-2*2 + 4*-1 + 6*4) = 4
    np.testing.assert_array_equal(orc.project(codes, s, g), [-10.5, 4.0])
    alpha = np.array([2.0, -4.0])
    base = np.array([10.0, 20.0, 30.0], dtype=np.float32)
    # w_r = base_r + 0.5*2*code[r,0] + 0.25*-4*code[r,1] = base + code0 - code1
    np.testing.assert_array_equal(orc.lift(codes, s, alpha, base), [13.0, 19.0, 19.0])
    P32 = np.array([[1, 0], [0, 2], [3, 0]], dtype=np.float32)
    np.testing.assert_array_equal(orc.project_f32(P32, g), [14.0, -2.0])
    np.testing.assert_array_equal(orc.lift_f32(P32, alpha, base), [12.0, 12.0, 36.0])


def test_projection_of_a_basis_column_is_a_gram_column_and_linearity():
    D, n = 600, 5
    _, _, codes, s = _quantised_basis(D, n, 8, seed=1)
    Pt = codes.astype(np.float64) * s.astype(np.float64)[None, :]
    G = Pt.T @ Pt
    for j in range(n):
        np.testing.assert_allclose(orc.project(codes, s, Pt[:, j]), G[:, j], rtol=1e-12)
    rng = np.random.default_rng(4)
    x, y = rng.standard_normal(D), rng.standard_normal(D)
    np.testing.assert_allclose(orc.project(codes, s, 2 * x - 3 * y),
                               2 * orc.project(codes, s, x) - 3 * orc.project(codes, s, y),
                               rtol=1e-10, atol=1e-12)


def test_alpha_zero_lifts_to_wbar_and_candidates_are_recovered():
    D, n = 900, 6
    A, P32, _, _ = _quantised_basis(D, n, 8, seed=2)
    wbar = orc.mean(A)
    np.testing.assert_array_equal(orc.lift_f32(P32, np.zeros(n), wbar), wbar)
    A64 = A.astype(np.float64)
    for i in range(n):
        # lift(project(w_i)) = w_i with no base, and around w_bar for the centred vector
        rec = orc.lift_f32(P32, orc.project_f32(P32, A64[:, i]), None)
        assert np.linalg.norm(rec - A64[:, i]) <= 1e-6 * np.linalg.norm(A64[:, i])   # float32 basis
        rec2 = orc.lift_f32(P32, orc.project_f32(P32, A64[:, i] - wbar), wbar)
        assert np.linalg.norm(rec2 - A64[:, i]) <= 1e-6 * np.linalg.norm(A64[:, i])


def test_update_rule_and_first_step_from_zero():
    c = np.array([1.0, -2.0, 0.5])
    np.testing.assert_allclose(orc.sgd_update(np.zeros(3), c, 0.1), -0.1 * c)
    a = np.array([1.0, 1.0, 1.0])
    # beta - eta (c + lambda beta)
    np.testing.assert_allclose(orc.sgd_update(a, c, 0.1, 0.5), a - 0.1 * (c + 0.5 * a), rtol=1e-15)


def test_step_equals_the_weight_space_recursion():
    """alpha-form (project, update, lift) against the weight-space form
    w <- (1 - eta*lambda) w - eta P P^T g of Section 4.2, for several steps."""
    D, n = 500, 4
    _, _, codes, s = _quantised_basis(D, n, 8, seed=3)
    Pt = codes.astype(np.float64) * s.astype(np.float64)[None, :]
    rng = np.random.default_rng(5)
    for lam in (0.0, 0.3):
        alpha = np.zeros(n)
        w_rec = np.zeros(D)                       # base 0: w = P beta
        for t in range(5):
            g = rng.standard_normal(D).astype(np.float32)
            alpha, w, c = orc.step(codes, s, g, alpha, np.zeros(D, dtype=np.float32), 0.05, lam)
            w_rec = (1 - 0.05 * lam) * w_rec - 0.05 * Pt @ (Pt.T @ g.astype(np.float64))
            np.testing.assert_allclose(w, w_rec, rtol=1e-10, atol=1e-13)
    # with a base point, w - w_bar follows the same recursion
    wbar = rng.standard_normal(D).astype(np.float32)
    alpha = np.zeros(n)
    dev = np.zeros(D)
    for t in range(3):
        g = rng.standard_normal(D).astype(np.float32)
        alpha, w, _ = orc.step(codes, s, g, alpha, wbar, 0.1, 0.0)
        dev = dev - 0.1 * Pt @ (Pt.T @ g.astype(np.float64))
        np.testing.assert_allclose(w - wbar.astype(np.float64), dev, rtol=1e-9, atol=1e-12)


def test_step_f32_matches_quantised_step_up_to_quantisation_error():
    D, n = 2000, 5
    _, P32, codes, s = _quantised_basis(D, n, 8, seed=6)
    rng = np.random.default_rng(6)
    g = rng.standard_normal(D).astype(np.float32)
    a1, w1, c1 = orc.step_f32(P32, g, np.zeros(n), np.zeros(D, dtype=np.float32), 0.1)
    a2, w2, c2 = orc.step(codes, s, g, np.zeros(n), np.zeros(D, dtype=np.float32), 0.1)
    assert np.linalg.norm(c1 - c2) <= 0.05 * np.linalg.norm(c1)
    assert np.linalg.norm(w1 - w2) <= 0.1 * np.linalg.norm(w1)


# ------------------------------------------------------------------ several gradients at once
def test_project_batch_brute_force_and_dense_product():
    # integers small enough for exact float64 arithmetic: a hand-computed 3 x 2 x 2 case
    codes = np.array([[1, -2], [3, 0], [-1, 4]], dtype=np.int8)
    s = np.array([0.5, 2.0], dtype=np.float32)
    G = np.array([[2.0, -1.0], [1.0, 0.0], [4.0, 3.0]], dtype=np.float32)
    # column 0: 0.5*(2+3-4)=0.5 ; 2*(-4+0+16)=24     column 1: 0.5*(-1+0-3)=-2 ; 2*(2+0+12)=28
    np.testing.assert_array_equal(orc.project_batch(codes, s, G), [[0.5, -2.0], [24.0, 28.0]])
    rng = np.random.default_rng(3)
    codes = rng.integers(-127, 128, size=(500, 7)).astype(np.int8)
    s = rng.random(7).astype(np.float32)
    G = rng.standard_normal((500, 5)).astype(np.float32)
    dense = (codes.astype(np.float64) * s.astype(np.float64)).T @ G.astype(np.float64)
    np.testing.assert_allclose(orc.project_batch(codes, s, G), dense, rtol=1e-12, atol=1e-12)
    # the projection of a sum of gradients is the sum of the columns (why accumulation needs no batch)
    np.testing.assert_allclose(orc.project(codes, s, G.astype(np.float64).sum(axis=1)),
                               orc.project_batch(codes, s, G).sum(axis=1), rtol=1e-11, atol=1e-11)
    # a transposed operand or a dropped scale fails: column b of G only meets column b of the result
    G2 = G.copy()
    G2[:, 3] = 0
    out = orc.project_batch(codes, s, G2)
    assert np.all(out[:, 3] == 0) and np.all(out[:, [0, 1, 2, 4]] == orc.project_batch(codes, s, G)[:, [0, 1, 2, 4]])


# ------------------------------------------------------------------ many steps in a row
def test_many_steps_end_at_the_projection_of_the_weighted_gradient_sum():
    """T steps of Algorithm 1's loop from alpha = 0 end at alpha_T = -eta P~^T G with
    G = sum_t (1 - eta*lambda)^(T-1-t) g_t, and w_T = w_bar + P~ alpha_T: the form the full-size
    sequence tests use where stepping the oracle through every gradient is out of reach."""
    from oracle_stream import weighted_gradient_sum
    D, n, T = 700, 6, 40
    _, _, codes, s = _quantised_basis(D, n, 8, seed=7)
    rng = np.random.default_rng(8)
    wbar = rng.standard_normal(D).astype(np.float32)
    for lr, lam in ((0.1, 0.0), (0.05, 0.3)):
        grads = [(rng.standard_normal(D) * 1e-3).astype(np.float32) for _ in range(T)]
        alpha = np.zeros(n)
        for g in grads:
            alpha, w, _ = orc.step(codes, s, g, alpha, wbar, lr, lam)
        G = weighted_gradient_sum(grads, lr, lam)
        a_lin = -lr * orc.project(codes, s, G)
        np.testing.assert_allclose(alpha, a_lin, rtol=1e-12, atol=1e-18)
        np.testing.assert_allclose(w, orc.lift(codes, s, a_lin, wbar), rtol=1e-13, atol=1e-15)
    # a dropped decay factor or a reversed order of the weights does not pass
    bad = np.zeros(D)
    for t, g in enumerate(grads):
        bad += (1.0 - 0.05 * 0.3) ** t * g.astype(np.float64)
    assert np.linalg.norm(-0.05 * orc.project(codes, s, bad) - alpha) > 1e-6 * np.linalg.norm(alpha)
