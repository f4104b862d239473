"""Pins for the oracle's per-column absmax quantiser and its byte layout."""

import os

import numpy as np

from oracle import twa_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _col(vals):
    return np.array(vals, dtype=np.float32).reshape(-1, 1)


def test_int8_hand_values_with_exact_ties():
    # absmax 127 -> scale exactly 1, so codes are the rounded values themselves
    P = _col([127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 2.0, -126.5, 126.49999, 0.0, 3.5])
    codes, s = orc.quantize(P, 8)
    assert s[0] == np.float32(1.0)
    # ties go to the even neighbour: 0.5->0, 1.5->2, 2.5->2, -0.5->0, -1.5->-2, -2.5->-2, 3.5->4
    np.testing.assert_array_equal(codes[:, 0], [127, 0, 2, 2, 0, -2, -2, 2, -126, 126, 0, 4])


def test_int4_hand_values_with_exact_ties():
    P = _col([7.0, 0.5, 1.5, 2.5, -3.5, -6.5, 6.5, -7.0, 6.4999995])
    codes, s = orc.quantize(P, 4)
    assert s[0] == np.float32(1.0)
    np.testing.assert_array_equal(codes[:, 0], [7, 0, 2, 2, -4, -6, 6, -7, 6])


def test_scale_is_float32_division_and_absmax_maps_to_qmax():
    rng = np.random.default_rng(1)
    P = rng.standard_normal((1000, 6)).astype(np.float32) * np.float32(3e-4)
    P[:, 4] = -np.abs(P[:, 4])                       # column whose absmax element is negative
    for bits, qmax in ((8, 127), (4, 7)):
        codes, s = orc.quantize(P, bits)
        for j in range(6):
            m = np.max(np.abs(P[:, j]))
            assert s[j] == np.float32(m) / np.float32(qmax)       # IEEE float32 division
            r = int(np.argmax(np.abs(P[:, j])))
            assert codes[r, j] == (qmax if P[r, j] > 0 else -qmax)
        assert codes.min() >= -qmax and codes.max() <= qmax        # -128 / -8 never produced
        # reconstruction error at most half a step (plus float32 rounding of the quotient)
        err = np.abs(P.astype(np.float64) - codes.astype(np.float64) * s.astype(np.float64))
        assert np.all(err <= 0.5 * s.astype(np.float64) * (1 + 1e-6))


def test_zero_column_and_single_row():
    P = np.zeros((5, 2), dtype=np.float32)
    P[:, 1] = [1, -2, 4, 0, 0.25]
    codes, s = orc.quantize(P, 8)
    assert s[0] == 0 and np.all(codes[:, 0] == 0)
    assert codes[2, 1] == 127 and codes[1, 1] == -64
    # -2/ (4/127) = -63.5 -> tie -> -64 (even)
    codes1, s1 = orc.quantize(_col([-3.0]), 4)
    assert codes1[0, 0] == -7 and s1[0] == np.float32(3.0) / np.float32(7.0)


def test_brute_force_matches_python_scalar_loop():
    rng = np.random.default_rng(2)
    P = (rng.standard_normal((64, 3)) * 0.01).astype(np.float32)
    for bits, qmax in ((8, 127), (4, 7)):
        codes, s = orc.quantize(P, bits)
        for j in range(3):
            m = max(abs(float(x)) for x in P[:, j])
            sj = np.float32(m) / np.float32(qmax)
            assert sj == s[j]
            for r in range(64):
                t = np.float32(P[r, j]) / sj                       # float32 division
                q = int(round(float(t)))                           # python round: ties to even
                q = max(-qmax, min(qmax, q))
                assert q == codes[r, j]


def test_pack_int4_bytes_by_hand_and_roundtrip():
    codes = np.array([[1], [-1], [7], [-7], [0], [-8 + 1], [3]], dtype=np.int8)   # D = 7 (odd)
    packed = orc.pack_codes(codes, 4)
    # (lo=1, hi=-1=0xF) (lo=7, hi=-7=0x9) (lo=0, hi=-7=0x9) (lo=3, hi=pad 0)
    np.testing.assert_array_equal(packed, np.array([[0xF1, 0x97, 0x90, 0x03]], dtype=np.uint8))
    np.testing.assert_array_equal(orc.unpack_codes(packed, 7, 4), codes)
    rng = np.random.default_rng(3)
    big = rng.integers(-7, 8, size=(101, 5)).astype(np.int8)
    np.testing.assert_array_equal(orc.unpack_codes(orc.pack_codes(big, 4), 101, 4), big)
    big8 = rng.integers(-127, 128, size=(33, 4)).astype(np.int8)
    p8 = orc.pack_codes(big8, 8)
    assert p8.shape == (4, 33) and p8[2, 5] == np.uint8(big8[5, 2])
    np.testing.assert_array_equal(orc.unpack_codes(p8, 33, 8), big8)


def test_storage_accounting_against_the_papers_tables():
    lines = [l.split() for l in open(os.path.join(GOLDEN, "paper_memory_ddp.txt"))
             if not l.startswith("#")]
    sgd_mb, fp32_mb, q4_mb = (float(x) for x in lines[0])
    D, n = (int(x) for x in lines[1])
    extra_fp32 = (fp32_mb - sgd_mb) * 1e6
    extra_q4 = (q4_mb - sgd_mb) * 1e6
    # the printed increments (+6000 MB, +750 MB) agree with 4nD and nBD/8 to a few per cent
    assert abs(orc.paper_storage_bytes(D, n, 32) - extra_fp32) / extra_fp32 < 0.05
    assert abs(orc.paper_storage_bytes(D, n, 4, L=161) - extra_q4) / extra_q4 < 0.05
    assert abs(extra_fp32 / extra_q4 - 8.0) < 1e-9                  # "around 8x"
    # the per-column format: same code bytes, 4n instead of 8L for the factors
    assert orc.storage_bytes(D, n, 32) == 4 * n * D
    assert orc.storage_bytes(D, n, 4) == n * D // 2 + 4 * n
    assert orc.storage_bytes(D, n, 8) == n * D + 4 * n
    assert orc.storage_bytes(7, 3, 4) == 3 * 4 + 12                  # odd D rounds each column up
    codes = np.zeros((7, 3), dtype=np.int8)
    assert orc.pack_codes(codes, 4).size + 4 * 3 == orc.storage_bytes(7, 3, 4)
    # k nodes hold ceil(n/k) columns each
    assert orc.paper_storage_bytes(D, 60, 32, k=4) == 4 * 15 * D
    assert orc.paper_storage_bytes(D, 10, 32, k=4) == 4 * 3 * D
