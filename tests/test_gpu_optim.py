"""GPU parity for the optimiser on the coefficients (Adam with decoupled decay inside the fused
step, per-column and layer-wise), the cosine schedule, and the fixed-weight averages."""

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
    x, y = np.asarray(x, dtype=np.float64), np.asarray(y, dtype=np.float64)
    return np.linalg.norm(x - y) / np.linalg.norm(y)


@pytest.mark.parametrize("bits", [32, 8, 4])
def test_step_adam_follows_the_oracle_over_iterations(env, bits):
    ctx, ws = env
    D, n = 70001, 33
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 5, DEV, ld=inputs.padded_ld(D, 4))
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    if bits == 32:
        P = P32
        Ph = W[:, :D].cpu().numpy().T
        proj = lambda g: orc.project_f32(Ph, g)
        lift = lambda a: orc.lift_f32(Ph, a, wbar.cpu().numpy())
    else:
        P = twa.twa_quantize_basis(ctx, P32, bits, ws)
        codes, s = twa.twa_basis_export(ctx, P)
        co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
        proj = lambda g: orc.project(co, so, g)
        lift = lambda a: orc.lift(co, so, a, wbar.cpu().numpy())
    alpha = torch.zeros(n, device=DEV)
    m = torch.zeros(n, device=DEV)
    v = torch.zeros(n, device=DEV)
    w = torch.empty(D, device=DEV)
    c = torch.empty(n, device=DEV)
    a_o, m_o, v_o = np.zeros(n), np.zeros(n), np.zeros(n)
    total = 6
    for t in range(1, total + 1):
        lr = twa.twa_cosine_lr(0.01, t - 1, total, 1e-4)
        assert abs(lr - orc.cosine_lr(0.01, t - 1, total, 1e-4)) <= 1e-9
        g = inputs.gradient(D, 1e-2, 3, t, torch.bfloat16, DEV)
        twa.twa_step_adam(ctx, P, g, lr, t, alpha, m, v, wbar, w, ws, beta1=0.9, beta2=0.98, eps=1e-9,
                          weight_decay=0.01, c_out=c)
        status_ok(ctx)
        c_o = proj(g.float().cpu().numpy())
        assert rel(c.cpu().numpy(), c_o) <= TOL
        # the oracle's optimiser on the GPU's own gradient and state of the previous step (float32 values)
        a_o, m_o, v_o = orc.adam_update(a_o, m_o, v_o, c.cpu().numpy(), lr, t, 0.9, 0.98, 1e-9, 0.01)
        # (the kernel updates from the unrounded c; sums of opposite signs in m bound the agreement by the
        # size of the terms, not of the result)
        np.testing.assert_allclose(alpha.cpu().numpy(), a_o, rtol=2e-6, atol=2e-6 * np.abs(a_o).max())
        np.testing.assert_allclose(m.cpu().numpy(), m_o, rtol=2e-6, atol=2e-6 * np.abs(m_o).max())
        np.testing.assert_allclose(v.cpu().numpy(), v_o, rtol=2e-6, atol=1e-30)
        assert rel(w.cpu().numpy(), lift(alpha.cpu().numpy().astype(np.float64))) <= TOL
        a_o, m_o, v_o = (x.cpu().numpy().astype(np.float64) for x in (alpha, m, v))
    # the first step moved every coefficient by about lr (sign step), unlike gradient descent
    assert np.all(np.abs(alpha.cpu().numpy()) > 0)


def test_layered_step_adam(env):
    ctx, _ = env
    D, n, layers = 70001, 20, [0, 64, 1000, 1001, 30000, 30017, 65536, 70001]
    L = len(layers) - 1
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 61, DEV, ld=inputs.padded_ld(D, 4))
    wbar = torch.empty(D, device=DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
    lb = twa.twa_quantize_affine(ctx, P32, layers, 4, lws)
    packed, a_g, b_g = twa.twa_layered_export(ctx, lb)
    b = packed.cpu().numpy()
    inter = np.empty((n, 2 * b.shape[1]), dtype=np.uint8)
    inter[:, 0::2], inter[:, 1::2] = b & 0xF, b >> 4
    codes = np.asfortranarray(inter[:, :D].T)
    a_h, b_h = a_g.cpu().numpy(), b_g.cpu().numpy()
    sws = twa.new_layered_step_workspace(lb)
    beta = torch.zeros((L, n), device=DEV)
    m = torch.zeros((L, n), device=DEV)
    v = torch.zeros((L, n), device=DEV)
    w = torch.empty(D, device=DEV)
    c = torch.empty((L, n), device=DEV)
    b_o, m_o, v_o = np.zeros((L, n)), np.zeros((L, n)), np.zeros((L, n))
    for t in range(1, 4):
        g = inputs.gradient(D, 1e-2, 8, t, torch.float32, DEV)
        twa.twa_layered_step_adam(ctx, lb, g, 0.01, t, beta, m, v, wbar, w, sws, weight_decay=0.01, c_out=c)
        status_ok(ctx)
        c_o = orc.project_layerwise(codes, layers, a_h, b_h, g.cpu().numpy())
        assert rel(c.cpu().numpy(), c_o) <= TOL
        b_o, m_o, v_o = orc.adam_update(b_o, m_o, v_o, c.cpu().numpy(), 0.01, t, weight_decay=0.01)
        np.testing.assert_allclose(beta.cpu().numpy(), b_o, rtol=2e-6, atol=2e-6 * np.abs(b_o).max())
        w_o = orc.lift_layerwise(codes, layers, a_h, b_h, beta.cpu().numpy(), wbar.cpu().numpy())
        assert rel(w.cpu().numpy(), w_o) <= TOL
        b_o, m_o, v_o = (x.cpu().numpy().astype(np.float64) for x in (beta, m, v))


def test_adam_rejects_bad_constants(env):
    ctx, ws = env
    D, n = 1000, 3
    P = torch.randn((n, inputs.padded_ld(D, 4)), device=DEV)
    P32 = twa.basis_from_tensor(P, D)
    z = torch.zeros(n, device=DEV)
    g = torch.zeros(D, device=DEV)
    w = torch.empty(D, device=DEV)
    for kw in ({"step": 0}, {"step": 1, "beta1": 1.0}, {"step": 1, "beta2": -0.1}, {"step": 1, "eps": -1.0}):
        step = kw.pop("step")
        with pytest.raises(twa.TwaError) as e:
            twa.twa_step_adam(ctx, P32, g, 0.01, step, z, z.clone(), z.clone(), w, w, ws, **kw)
        assert e.value.code == twa.TWA_ERR_INVALID_ARG


@pytest.mark.parametrize("D,n", [(5, 2), (70001, 10), (300007, 50)])
def test_weighted_average_swa_lawa_ema(env, D, n):
    ctx, ws = env
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 7, DEV, ld=inputs.padded_ld(D, 4))
    A = W[:, :D].cpu().numpy().T
    out = torch.empty(D, device=DEV)
    t_last = max(1, n // 3)
    d = 0.9
    ema = np.array([d ** (n - 1)] + [(1 - d) * d ** (n - 1 - i) for i in range(1, n)])
    for wts in (np.full(n, 1.0 / n), np.r_[np.zeros(n - t_last), np.full(t_last, 1.0 / t_last)], ema):
        wt = torch.tensor(wts, dtype=torch.float32, device=DEV)
        twa.twa_weighted_average(ctx, W, D, wt, out, ws)
        status_ok(ctx)
        ref = orc.weighted_average(A, wt.cpu().numpy())
        assert rel(out.cpu().numpy(), ref) <= TOL
        assert np.max(np.abs(out.cpu().numpy() - ref)) <= 8 * np.spacing(np.float32(np.abs(ref).max())) * np.sqrt(n)
    # equal weights agree with the library's own mean kernel to float32 rounding
    wbar = torch.empty(D, device=DEV)
    twa.twa_mean(ctx, W, D, wbar)
    twa.twa_weighted_average(ctx, W, D, torch.full((n,), 1.0 / n, device=DEV), out, ws)
    assert rel(out.cpu().numpy(), wbar.cpu().numpy()) <= 1e-6
    assert torch.equal(W[:, :D].cpu(), torch.from_numpy(np.ascontiguousarray(A.T)))       # candidates untouched
