"""Pins for the oracle's version of the paper's default construction: decentralise +
normalise per layer, per-layer min-max B-bit codes, layer-wise coefficients."""

import numpy as np

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import inputs

LAYERS = [0, 7, 300, 301, 1000, 1777]


def _cands(D=1777, n=6, seed=0):
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, seed, "cpu")
    return W[:, :D].numpy().T


def test_center_normalize_closed_form_and_invariants():
    # two layers, three candidates with hand-checkable numbers
    W = np.array([[1, 3, 5], [2, 2, 2], [0, 3, 6], [1, 1, 4]], dtype=np.float32)
    P, wbar = orc.center_normalize(W, [0, 2, 4])
    np.testing.assert_allclose(wbar, [3, 2, 3, 2])
    # layer 0: rows 0-1 centred = [[-2,0,2],[0,0,0]] -> unit vectors (-1,0), 0, (1,0)
    np.testing.assert_allclose(P[:2], [[-1, 0, 1], [0, 0, 0]], atol=1e-15)
    # layer 1: centred rows [[-3,0,3],[-1,-1,2]]: column 0 = (-3,-1)/sqrt(10)
    np.testing.assert_allclose(P[2:, 0], np.array([-3, -1]) / np.sqrt(10), atol=1e-15)
    np.testing.assert_allclose(P[2:, 1], [0, -1], atol=1e-15)
    A = _cands()
    P, wbar = orc.center_normalize(A, LAYERS)
    np.testing.assert_allclose(wbar, A.astype(np.float64).mean(axis=1), rtol=1e-14)
    for l in range(len(LAYERS) - 1):
        blk = P[LAYERS[l]:LAYERS[l + 1]]
        np.testing.assert_allclose(np.linalg.norm(blk, axis=0), 1.0, rtol=1e-12)       # unit per layer
        # the centred candidates sum to zero: sum_i ||w_i^l - w_bar^l|| e_i^l = 0
        norms = np.linalg.norm(A[LAYERS[l]:LAYERS[l + 1]].astype(np.float64)
                               - A[LAYERS[l]:LAYERS[l + 1]].astype(np.float64).mean(axis=1, keepdims=True), axis=0)
        assert np.max(np.abs(blk @ norms)) <= 1e-12 * norms.max()
    # one layer over everything = the paper's whole-vector formula
    P1, _ = orc.center_normalize(A, [0, A.shape[0]])
    V = A.astype(np.float64) - wbar[:, None]
    np.testing.assert_allclose(P1, V / np.linalg.norm(V, axis=0), atol=1e-14)
    # columns are not orthogonal (the paper reports a residual correlation) but far from parallel
    C = P1.T @ P1
    assert np.max(np.abs(C - np.diag(np.diag(C)))) < 0.95


def test_candidate_equal_to_the_mean_gives_a_zero_direction():
    W = np.array([[1, 1, 1], [2, 4, 6]], dtype=np.float32)       # layer 0 (row 0) is identical in all candidates
    P, _ = orc.center_normalize(W, [0, 1, 2])
    np.testing.assert_array_equal(P[0], [0, 0, 0])
    np.testing.assert_allclose(P[1], [-1, 0, 1])


def test_affine_hand_values_ties_and_range():
    # one layer, values chosen so that a = 1 and b = -2 exactly at 4 bits: range [-2, 13]
    P = np.array([[-2.0, 13.0], [0.5, -1.5], [2.5, 3.5], [12.5, 0.0]], dtype=np.float32)
    codes, a, b = orc.affine_quantize(P, [0, 4], 4)
    assert a[0] == 1.0 and b[0] == -2.0
    # (p - b)/a = p + 2: 0, 15, 2.5->2, 0.5->0, 4.5->4, 5.5->6, 14.5->14, 2
    np.testing.assert_array_equal(codes, [[0, 15], [2, 0], [4, 6], [14, 2]])
    rng = np.random.default_rng(0)
    P = (rng.standard_normal((500, 5)) * 0.01).astype(np.float32)
    layers = [0, 100, 101, 500]
    for bits in (8, 4, 2, 1):
        codes, a, b = orc.affine_quantize(P, layers, bits)
        top = 2 ** bits - 1
        assert codes.min() == 0 and codes.max() == top
        for l in range(3):
            blk = P[layers[l]:layers[l + 1]]
            assert b[l] == blk.min()
            assert a[l] == np.float32(np.float32(blk.max() - blk.min()) / np.float32(top))
            r, c = np.unravel_index(np.argmax(blk), blk.shape)
            assert codes[layers[l] + r, c] == top                     # the maximum maps to the top level
            r, c = np.unravel_index(np.argmin(blk), blk.shape)
            assert codes[layers[l] + r, c] == 0
        deq = orc.affine_dequantize(codes, layers, a, b)
        step = np.repeat(a.astype(np.float64), np.diff(layers))[:, None]
        assert np.all(np.abs(deq - P) <= 0.5 * step * (1 + 1e-5) + 1e-12)   # half a step
    # brute force, scalar python, on a tiny block
    blk = P[:7, :2]
    codes, a, b = orc.affine_quantize(blk, [0, 7], 4)
    for r in range(7):
        for c in range(2):
            t = np.float32(np.float32(blk[r, c] - b[0]) / a[0])
            assert codes[r, c] == max(0, min(15, int(round(float(t)))))


def test_constant_layer_and_storage_formula():
    P = np.full((4, 3), 0.25, dtype=np.float32)
    codes, a, b = orc.affine_quantize(P, [0, 4], 4)
    assert a[0] == 0 and b[0] == np.float32(0.25) and not codes.any()
    np.testing.assert_allclose(orc.affine_dequantize(codes, [0, 4], a, b), 0.25)
    # the paper's accounting: n*B*D/8 + 8L; 32/B compression against float32 up to the factors
    D, n, L = 25557032, 60, 161
    assert orc.paper_affine_storage_bytes(D, n, 4, L) == n * D / 2 + 8 * L
    assert abs(4 * n * D / orc.paper_affine_storage_bytes(D, n, 4, L) - 8.0) < 1e-4


def test_layerwise_project_lift_equal_block_diagonal_dense_algebra():
    A = _cands()
    D, n = A.shape
    P, wbar = orc.center_normalize(A, LAYERS)
    P32 = np.asfortranarray(P.astype(np.float32))
    rng = np.random.default_rng(1)
    g = rng.standard_normal(D).astype(np.float32)
    L = len(LAYERS) - 1
    beta = rng.standard_normal((L, n))
    for bits in (8, 4):
        codes, a, b = orc.affine_quantize(P32, LAYERS, bits)
        Pt = orc.affine_dequantize(codes, LAYERS, a, b)
        c = orc.project_layerwise(codes, LAYERS, a, b, g)
        w = orc.lift_layerwise(codes, LAYERS, a, b, beta, wbar.astype(np.float32))
        for l in range(L):
            r0, r1 = LAYERS[l], LAYERS[l + 1]
            np.testing.assert_allclose(c[l], Pt[r0:r1].T @ g[r0:r1].astype(np.float64), rtol=1e-11, atol=1e-14)
            np.testing.assert_allclose(w[r0:r1], wbar.astype(np.float32)[r0:r1].astype(np.float64)
                                       + Pt[r0:r1] @ beta[l], rtol=1e-11, atol=1e-14)
        # beta = 0 lifts to the base point; one layer with L = 1 equals the whole-vector step
        np.testing.assert_array_equal(orc.lift_layerwise(codes, LAYERS, a, b, np.zeros((L, n)), wbar), wbar)
    codes1, a1, b1 = orc.affine_quantize(P32, [0, D], 8)
    Pt1 = orc.affine_dequantize(codes1, [0, D], a1, b1)
    np.testing.assert_allclose(orc.project_layerwise(codes1, [0, D], a1, b1, g)[0], Pt1.T @ g.astype(np.float64),
                               rtol=1e-11)


def test_layerwise_step_equals_per_layer_weight_space_recursion():
    A = _cands(seed=3)
    D, n = A.shape
    P, wbar = orc.center_normalize(A, LAYERS)
    codes, a, b = orc.affine_quantize(np.asfortranarray(P.astype(np.float32)), LAYERS, 4)
    Pt = orc.affine_dequantize(codes, LAYERS, a, b)
    L = len(LAYERS) - 1
    rng = np.random.default_rng(2)
    for lam in (0.0, 0.2):
        beta = np.zeros((L, n))
        dev = np.zeros(D)
        for t in range(4):
            g = rng.standard_normal(D).astype(np.float32)
            beta, w, c = orc.step_layerwise(codes, LAYERS, a, b, g, beta, np.zeros(D, dtype=np.float32), 0.05, lam)
            for l in range(L):
                r0, r1 = LAYERS[l], LAYERS[l + 1]
                dev[r0:r1] = (1 - 0.05 * lam) * dev[r0:r1] - 0.05 * Pt[r0:r1] @ (Pt[r0:r1].T @ g[r0:r1].astype(np.float64))
            np.testing.assert_allclose(w, dev, rtol=1e-9, atol=1e-12)
    c0 = orc.project_layerwise(codes, LAYERS, a, b, g)
    np.testing.assert_allclose(orc.step_layerwise(codes, LAYERS, a, b, g, np.zeros((L, n)), wbar, 0.1)[0], -0.1 * c0)


def test_unsigned_packing_hand_bytes_and_roundtrip():
    """The canonical image of unsigned B-bit codes, against bytes worked out by hand."""
    codes = np.array([[1, 0], [0, 1], [1, 1], [1, 0], [0, 0], [0, 1], [1, 0], [1, 1], [1, 1]], dtype=np.uint8)
    # 1 bit, column 0 rows 0..8 = 1,0,1,1,0,0,1,1 | 1  -> bits 0,2,3,6,7 = 0xCD, then 0x01
    np.testing.assert_array_equal(orc.pack_unsigned(codes, 1), [[0xCD, 0x01], [0xA6, 0x01]])
    c2 = np.array([[3], [0], [2], [1], [1]], dtype=np.uint8)
    # 2 bits: 3 | 0<<2 | 2<<4 | 1<<6 = 0x63, then 0x01
    np.testing.assert_array_equal(orc.pack_unsigned(c2, 2), [[0x63, 0x01]])
    c3 = np.array([[7], [5], [2]], dtype=np.uint8)
    # 3-bit codes in 4-bit slots: 7 | 5<<4 = 0x57, then 0x02
    np.testing.assert_array_equal(orc.pack_unsigned(c3, 3), [[0x57, 0x02]])
    np.testing.assert_array_equal(orc.pack_unsigned(c3, 4), [[0x57, 0x02]])
    np.testing.assert_array_equal(orc.pack_unsigned(c3, 8), [[7, 5, 2]])
    c16 = np.array([[0x1234], [0xFFFF], [7]], dtype=np.uint16)
    np.testing.assert_array_equal(orc.pack_unsigned(c16, 16), [[0x34, 0x12, 0xFF, 0xFF, 0x07, 0x00]])
    rng = np.random.default_rng(11)
    for bits in (1, 2, 3, 4, 8, 16):
        for D in (1, 7, 8, 9, 1001):
            c = rng.integers(0, 2 ** bits, size=(D, 3)).astype(np.uint16)
            p = orc.pack_unsigned(c, bits)
            assert p.shape == (3, (D * orc.SLOT_BITS[bits] + 7) // 8)
            np.testing.assert_array_equal(orc.unpack_unsigned(p, D, bits), c)


def test_affine_quantiser_at_every_width_of_the_ablation():
    """B in {1, 2, 3, 4, 8, 16} (the paper's bits ablation): codes stay in range, the half-step
    bound holds, and a two-level layer at 1 bit maps its minimum to 0 and its maximum to 1."""
    rng = np.random.default_rng(5)
    P = rng.standard_normal((500, 4)).astype(np.float32)
    for bits in (1, 2, 3, 4, 8, 16):
        codes, a, b = orc.affine_quantize(P, [0, 200, 500], bits)
        assert codes.max() <= 2 ** bits - 1 and codes.min() >= 0
        deq = orc.affine_dequantize(codes, [0, 200, 500], a, b)
        step = np.repeat(a.astype(np.float64), [200, 300])[:, None]
        # half a step, plus the float32 roundings of the subtraction and of the quotient
        assert np.all(np.abs(deq - P) <= 0.5 * step + 8 * np.finfo(np.float32).eps * np.abs(P).max())
    two = np.array([[-1.0], [3.0], [3.0], [-1.0]], dtype=np.float32)
    codes, a, b = orc.affine_quantize(two, [0, 4], 1)
    assert a[0] == 4.0 and b[0] == -1.0
    np.testing.assert_array_equal(codes[:, 0], [0, 1, 1, 0])
