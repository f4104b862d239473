"""GPU parity for the paper's default construction: decentralise + normalise per layer, per-layer
min-max B-bit codes (bit-exact against the oracle on the GPU's own float32 basis)."""

import numpy as np
import pytest
import torch

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import inputs, twa

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-5


@pytest.fixture(scope="module")
def env():
    torch.cuda.set_device(0)
    ctx = twa.twa_create(0)
    ws = twa.new_workspace(DEV)
    yield ctx, ws
    torch.cuda.synchronize()
    twa.twa_destroy(ctx)


def status_ok(ctx):
    code, detail = twa.twa_get_status(ctx)
    assert code == 0, (twa.twa_strerror(code), detail)


def rel(x, y):
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    return np.linalg.norm(x - y) / np.linalg.norm(y)


def unpack_unsigned(packed, D, bits):
    packed = packed.astype(np.uint8)
    if bits == 8:
        return np.asfortranarray(packed[:, :D].T)
    lo, hi = packed & 0xF, packed >> 4
    inter = np.empty((packed.shape[0], 2 * packed.shape[1]), dtype=np.uint8)
    inter[:, 0::2], inter[:, 1::2] = lo, hi
    return np.asfortranarray(inter[:, :D].T)


CASES = [
    (1777, 6, [0, 7, 300, 301, 1000, 1777]),
    (70001, 33, [0, 64, 1000, 1001, 30000, 30017, 65536, 70001]),
    (300000, 20, [0, 300000]),
    (5, 2, [0, 1, 5]),
]


@pytest.mark.parametrize("D,n,layers", CASES)
def test_build_centered(env, D, n, layers):
    ctx, _ = env
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 41, DEV, ld=inputs.padded_ld(D, 4))
    A = W[:, :D].cpu().numpy().T.copy()
    wbar = torch.empty(D, device=DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
    status_ok(ctx)
    P_o, wbar_o = orc.center_normalize(A, layers)
    np.testing.assert_array_equal(wbar.cpu().numpy(), wbar_o.astype(np.float32))
    Pg = W[:, :D].cpu().numpy().T
    # float32 rounding of the candidates' difference from the mean limits the agreement
    scale = np.abs(A).max()
    for l in range(len(layers) - 1):
        r0, r1 = layers[l], layers[l + 1]
        norms = np.linalg.norm(A[r0:r1].astype(np.float64) - wbar_o[r0:r1, None], axis=0)
        tol = 4 * np.finfo(np.float32).eps * np.maximum(1.0, scale * np.sqrt(r1 - r0) / np.maximum(norms, 1e-300))
        assert np.all(np.abs(Pg[r0:r1] - P_o[r0:r1]).max(axis=0) <= tol)
    assert torch.all(W[:, D:] == 0)
    assert (P32.D, P32.n, P32.bits) == (D, n, 32)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("D,n,layers", CASES)
def test_quantize_affine_bit_exact(env, D, n, layers, bits):
    ctx, _ = env
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 42, DEV, ld=inputs.padded_ld(D, 4))
    wbar = torch.empty(D, device=DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
    if len(layers) > 3:
        W[:, layers[1]:layers[2]] = 0.125                      # a constant layer: a = 0
    lb = twa.twa_quantize_affine(ctx, P32, layers, bits, lws)
    status_ok(ctx)
    codes_g, a_g, b_g = twa.twa_layered_export(ctx, lb)
    Pg = np.asfortranarray(W[:, :D].cpu().numpy().T)
    codes_o, a_o, b_o = orc.affine_quantize(Pg, layers, bits)
    np.testing.assert_array_equal(a_g.cpu().numpy(), a_o)
    np.testing.assert_array_equal(b_g.cpu().numpy(), b_o)
    np.testing.assert_array_equal(unpack_unsigned(codes_g.cpu().numpy(), D, bits), codes_o)
    assert lb.desc.codes.D == twa.twa_layered_rows(layers, bits)
    # storage: n*B*D/8 code bytes (+ per-layer padding to 64-byte granules) and two factors per layer
    assert codes_g.numel() == n * ((D * bits + 7) // 8)


def test_affine_nonfinite_is_reported(env):
    ctx, _ = env
    D, n, layers = 5000, 3, [0, 100, 5000]
    P = torch.randn((n, D), device=DEV)
    P[1, 4000] = float("nan")
    lws = twa.new_layered_workspace(layers, n, DEV)
    twa.twa_quantize_affine(ctx, twa.basis_from_tensor(P, D), layers, 4, lws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_NONFINITE, 1)
    twa.twa_clear_status(ctx)
