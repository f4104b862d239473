"""Seeded random shapes through the whole path: n from 1 to 128 around the kernels' internal group
sizes (8, 16, 32, 64), D from n to 250,000 rows with every kind of ragged tail, random layer cuts
(one-row layers, neighbouring cuts) and every code width.  Each case checks what the fixed-shape tests
check -- mean, orthonormality, codes and scales bit-exact against the oracle's quantiser on the
library's own float32 basis, projection (single, batched, float32 basis) and lift within the bounds --
so that a shape nobody thought of listing still meets the oracle."""

import numpy as np
import pytest
import torch

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import inputs, twa

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-5
N_CHOICES = [1, 2, 3, 7, 8, 9, 15, 16, 17, 24, 31, 32, 33, 50, 63, 64, 65, 100, 127, 128]


@pytest.fixture(scope="module")
def env():
    torch.cuda.set_device(0)
    ctx = twa.twa_create(0)
    ws = twa.new_workspace(DEV)
    yield ctx, ws
    torch.cuda.synchronize()
    twa.twa_destroy(ctx)


def status_ok(ctx, tag):
    code, detail = twa.twa_get_status(ctx)
    assert code == 0, (twa.twa_strerror(code), detail, tag)


def rel(x, y):
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    return np.linalg.norm(x - y) / np.linalg.norm(y)


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_per_column(env, seed):
    ctx, ws = env
    rng = np.random.default_rng(1000 + seed)
    for case in range(8):
        n = int(rng.choice(N_CHOICES))
        D = int(rng.integers(n, 250000))
        if rng.random() < 0.3:
            D = max(n, D // 100)
        tag = f"seed={seed} case={case} D={D} n={n}"
        W = inputs.trajectory_candidates(D, n, 0.005, 0.001, int(rng.integers(1 << 30)), DEV, ld=inputs.padded_ld(D, 4))
        A = W[:, :D].cpu().numpy().T.copy()
        wbar = torch.empty(D, device=DEV)
        P32, (q8, q4) = twa.twa_build_quantized(ctx, W, D, wbar, [8, 4], ws)
        status_ok(ctx, tag)
        Pg = W[:, :D].cpu().numpy().T
        P64 = Pg.astype(np.float64)
        assert np.max(np.abs(P64.T @ P64 - np.eye(n))) <= 1e-5, tag
        np.testing.assert_array_equal(wbar.cpu().numpy(), orc.mean(A).astype(np.float32), err_msg=tag)
        gdt = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        gen = torch.Generator(device=DEV).manual_seed(seed * 100 + case)
        g = (torch.randn(D, generator=gen, device=DEV) * 1e-3).to(gdt)
        g_h = g.float().cpu().numpy()
        alpha = torch.randn(n, generator=gen, device=DEV)
        for bits, q in ((8, q8), (4, q4)):
            codes, s = twa.twa_basis_export(ctx, q)
            co, so = orc.quantize(np.asfortranarray(Pg), bits)
            np.testing.assert_array_equal(s.cpu().numpy(), so, err_msg=tag)
            np.testing.assert_array_equal(codes.cpu().numpy(), orc.pack_codes(co, bits), err_msg=tag)
            # |c_j - c_j(oracle)| <= 1e-5 |p~_j| |g|: a single coefficient may be small by cancellation
            pn = so.astype(np.float64) * np.linalg.norm(co.astype(np.float64), axis=0)
            c, w = torch.empty(n, device=DEV), torch.empty(D, device=DEV)
            twa.twa_project(ctx, q, g, c, ws)
            twa.twa_lift(ctx, q, alpha, wbar, w, ws)
            c_o = orc.project(co, so, g_h)
            assert np.all(np.abs(c.cpu().numpy() - c_o) <= TOL * pn * np.linalg.norm(g_h) + 1e-30), (bits, tag)
            assert rel(w.cpu().numpy(), orc.lift(co, so, alpha.cpu().numpy(), wbar.cpu().numpy())) <= TOL, (bits, tag)
            batch = int(rng.integers(1, 12))
            G = (torch.randn((batch, inputs.padded_ld(D, 8)), generator=gen, device=DEV) * 1e-3).to(gdt)
            C = torch.empty((batch, n), device=DEV)
            twa.twa_project_batch(ctx, q, G, C, ws)
            G_h = G[:, :D].float().cpu().numpy()
            C_o = orc.project_batch(co, so, G_h.T).T
            for b in range(batch):
                assert np.all(np.abs(C[b].cpu().numpy() - C_o[b]) <= TOL * pn * np.linalg.norm(G_h[b]) + 1e-30), (bits, b, tag)
        c = torch.empty(n, device=DEV)
        twa.twa_project(ctx, P32, g, c, ws)
        assert np.all(np.abs(c.cpu().numpy() - orc.project_f32(Pg, g_h)) <= TOL * np.linalg.norm(g_h)), tag
        status_ok(ctx, tag)


def _term_scale(codes, layers, a, b, g64):
    L, n = len(layers) - 1, codes.shape[1]
    s = np.zeros((L, n))
    ag = np.abs(g64)
    for l in range(L):
        r0, r1 = layers[l], layers[l + 1]
        s[l] = abs(float(a[l])) * (codes[r0:r1].astype(np.float64).T @ ag[r0:r1]) + abs(float(b[l])) * ag[r0:r1].sum()
    return s


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_layer_wise(env, seed):
    ctx, _ = env
    rng = np.random.default_rng(2000 + seed)
    for case in range(8):
        bits = int(rng.choice([8, 4, 3, 2, 1, 16]))
        n = int(rng.choice([1, 2, 5, 8, 17, 32, 33, 50, 64, 100, 128]))
        if bits == 16:
            n = min(n, 64)
        D = int(rng.integers(max(n, 2), 120000))
        L = int(rng.integers(1, 9))
        cuts = sorted(set(int(x) for x in rng.integers(1, D, size=L - 1))) if L > 1 else []
        if cuts and rng.random() < 0.5:
            cuts = sorted(set(cuts + [min(D - 1, cuts[0] + 1)]))       # a one-row layer
        layers = [0] + cuts + [D]
        tag = f"seed={seed} case={case} D={D} n={n} bits={bits} layers={layers}"
        W = inputs.trajectory_candidates(D, n, 0.005, 0.001, int(rng.integers(1 << 30)), DEV, ld=inputs.padded_ld(D, 4))
        A = W[:, :D].cpu().numpy().T.copy()
        wbar = torch.empty(D, device=DEV)
        lws = twa.new_layered_workspace(layers, n, DEV)
        P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
        lb = twa.twa_quantize_affine(ctx, P32, layers, bits, lws)
        status_ok(ctx, tag)
        cg, ag, bg = twa.twa_layered_export(ctx, lb)
        co, ao, bo = orc.affine_quantize(np.asfortranarray(W[:, :D].cpu().numpy().T), layers, bits)
        np.testing.assert_array_equal(ag.cpu().numpy(), ao, err_msg=tag)
        np.testing.assert_array_equal(bg.cpu().numpy(), bo, err_msg=tag)
        np.testing.assert_array_equal(orc.unpack_unsigned(cg.cpu().numpy(), D, bits), co, err_msg=tag)
        # the row-chunked build of the same candidates: codes are the quantiser of its own float32 vectors
        chunk_rows = int(rng.choice([1024, 4096, 8192, 65536]))
        lb2 = twa.twa_layered_build_begin(ctx, D, n, layers, bits, lws, DEV)
        wbar2 = torch.empty(D, device=DEV)
        q32 = torch.zeros((n, inputs.padded_ld(D, 4)), device=DEV)
        At = torch.from_numpy(np.ascontiguousarray(A.T)).to(DEV)
        for p in range(3):
            for r0 in range(0, D, chunk_rows):
                rows = min(chunk_rows, D - r0)
                buf = torch.zeros((n, inputs.padded_ld(rows, 4)), device=DEV)
                buf[:, :rows] = At[:, r0:r0 + rows]
                twa.twa_layered_build_feed(ctx, lb2, p, buf, r0, rows, wbar2, lws,
                                           q32_out=q32[:, r0:r0 + rows] if p == 1 else None)
            twa.twa_layered_build_end_pass(ctx, lb2, p, lws)
        status_ok(ctx, tag)
        assert torch.equal(wbar, wbar2), tag
        c2, a2, b2 = twa.twa_layered_export(ctx, lb2)
        co2, ao2, bo2 = orc.affine_quantize(np.asfortranarray(q32[:, :D].cpu().numpy().T), layers, bits)
        np.testing.assert_array_equal(a2.cpu().numpy(), ao2, err_msg=tag)
        np.testing.assert_array_equal(b2.cpu().numpy(), bo2, err_msg=tag)
        np.testing.assert_array_equal(orc.unpack_unsigned(c2.cpu().numpy(), D, bits), co2, err_msg=tag)
        # projection and lift on the resident basis
        sws = twa.new_layered_step_workspace(lb)
        gdt = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        g = inputs.gradient(D, 1e-3, 7, seed * 100 + case, gdt, DEV)
        Ln = len(layers) - 1
        c = torch.empty((Ln, n), device=DEV)
        twa.twa_layered_project(ctx, lb, g, c, sws)
        g64 = g.float().cpu().numpy().astype(np.float64)
        c_o = orc.project_layerwise(co, layers, ao, bo, g64)
        assert np.all(np.abs(c.cpu().numpy() - c_o) <= 2e-6 * _term_scale(co, layers, ao, bo, g64) + 1e-30), tag
        gen = torch.Generator(device=DEV).manual_seed(seed * 100 + case)
        beta = torch.randn((Ln, n), generator=gen, device=DEV) * 0.3
        w = torch.empty(D, device=DEV)
        twa.twa_layered_lift(ctx, lb, beta, wbar, w, sws)
        w_o = orc.lift_layerwise(co, layers, ao, bo, beta.cpu().numpy(), wbar.cpu().numpy())
        assert rel(w.cpu().numpy(), w_o) <= TOL, tag
        status_ok(ctx, tag)


@pytest.mark.parametrize("seed", range(4))
def test_random_shapes_walked_in_slabs(seed):
    """TWA_TUNE_SLAB_ROWS makes the stepping calls walk a basis in slabs of 65536 k rows -- the walk every
    basis above 2^31 - 2^20 rows gets -- so that random shapes meet it: D on, just past and far from a slab
    boundary, 2 to 16 slabs, 8-bit, 4-bit and float32 bases.  The lift must equal the one-launch lift bit
    for bit (rows do not interact); projection, SGD step and Adam step must meet the oracle within the
    bounds of the one-launch calls and the one-launch result to rounding; so must the batched projection."""
    torch.cuda.set_device(0)
    ctx, ref = twa.twa_create(0), twa.twa_create(0)
    ws, ws_ref = twa.new_workspace(DEV), twa.new_workspace(DEV)
    rng = np.random.default_rng(4000 + seed)
    for case in range(6):
        n = int(rng.choice(N_CHOICES))
        slab = 65536 * int(rng.integers(1, 4))
        slabs = int(rng.integers(2, 17))
        tail = int(rng.choice([0, 1, 2, 511, 512, 1023, 4097, slab - 1, int(rng.integers(1, slab))]))
        D = slab * (slabs - 1) + (tail if tail else slab)
        bits = int(rng.choice([8, 4, 32]))
        tag = f"seed={seed} case={case} D={D} n={n} bits={bits} slab={slab}"
        gen = torch.Generator(device=DEV).manual_seed(seed * 100 + case)
        P = torch.zeros((n, inputs.padded_ld(D, 4)), device=DEV)
        P[:, :D] = torch.randn((n, D), generator=gen, device=DEV) / np.sqrt(D)
        B = twa.basis_from_tensor(P, D)
        if bits != 32:
            B = twa.twa_quantize_basis(ref, B, bits, ws_ref)
            codes, s = twa.twa_basis_export(ref, B)
            co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
        else:
            P_h = P[:, :D].cpu().numpy().T
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_SLAB_ROWS, slab)
        gdt = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        g = (torch.randn(D, generator=gen, device=DEV) * 1e-3).to(gdt)
        g_h = g.float().cpu().numpy()
        wbar = torch.randn(D, generator=gen, device=DEV)
        # projection
        c, c1 = torch.empty(n, device=DEV), torch.empty(n, device=DEV)
        twa.twa_project(ctx, B, g, c, ws)
        twa.twa_project(ref, B, g, c1, ws_ref)
        c_o = orc.project(co, so, g_h) if bits != 32 else orc.project_f32(P_h, g_h)
        g_norm = np.linalg.norm(g_h.astype(np.float64))
        p_norm = (np.linalg.norm(co.astype(np.float64), axis=0) * np.abs(so) if bits != 32
                  else np.linalg.norm(P_h.astype(np.float64), axis=0))
        assert np.all(np.abs(c.cpu().numpy() - c_o) <= TOL * p_norm * g_norm + 1e-30), tag
        assert np.all(np.abs(c.cpu().numpy() - c1.cpu().numpy()) <= 2e-6 * p_norm * g_norm + 1e-30), tag
        # several gradients per projection: every slab after the first adds to the results
        batch = int(rng.integers(1, 11))
        G = torch.zeros((batch, inputs.padded_ld(D, 8)), dtype=gdt, device=DEV)
        G[:, :D] = (torch.randn((batch, D), generator=gen, device=DEV) * 1e-3).to(gdt)
        C = torch.full((batch, n), 7.0, device=DEV)
        twa.twa_project_batch(ctx, B, G, C, ws)
        for b_ in range(batch):
            gb = G[b_, :D].float().cpu().numpy()
            cb = orc.project(co, so, gb) if bits != 32 else orc.project_f32(P_h, gb)
            bound = TOL * p_norm * np.linalg.norm(gb.astype(np.float64)) + 1e-30
            assert np.all(np.abs(C[b_].cpu().numpy() - cb) <= bound), (tag, b_)
        # lift: bit for bit the one-launch lift, with and without the base point
        alpha = torch.randn(n, generator=gen, device=DEV)
        w, w1 = torch.empty(D, device=DEV), torch.empty(D, device=DEV)
        for base in (wbar, None):
            twa.twa_lift(ctx, B, alpha, base, w, ws)
            twa.twa_lift(ref, B, alpha, base, w1, ws_ref)
            assert torch.equal(w, w1), tag
        # SGD step and Adam step from zero state
        a, a1 = torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
        twa.twa_step(ctx, B, g, 0.1, 0.01, a, wbar, w, ws, c_out=c)
        a_o = orc.sgd_update(np.zeros(n), c_o, 0.1, 0.01)
        assert np.all(np.abs(a.cpu().numpy() - a_o) <= 0.1 * TOL * p_norm * g_norm + 1e-30), tag
        twa.twa_lift(ref, B, a, wbar, w1, ws_ref)
        assert torch.equal(w, w1), tag
        m, v = torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
        twa.twa_step_adam(ctx, B, g, 1e-2, 1, a1, m, v, wbar, w, ws, weight_decay=0.01)
        _, m_o, v_o = orc.adam_update(np.zeros(n), np.zeros(n), np.zeros(n), c_o, 1e-2, 1, weight_decay=0.01)
        assert np.all(np.abs(m.cpu().numpy() - m_o) <= 0.1 * TOL * p_norm * g_norm + 1e-30), tag
        assert rel(v.cpu().numpy(), v_o) <= 1e-3, tag
        twa.twa_lift(ref, B, a1, wbar, w1, ws_ref)
        assert torch.equal(w, w1), tag
        status_ok(ctx, tag)
        status_ok(ref, tag)
    # more than sixteen slabs do not fit the workspace's slots: refused on the host
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_SLAB_ROWS, 65536)
    Pbig = torch.zeros((1, 65536 * 16 + 4), device=DEV)
    with pytest.raises(twa.TwaError):
        twa.twa_project(ctx, twa.basis_from_tensor(Pbig, 65536 * 16 + 1), torch.zeros(65536 * 16 + 4, device=DEV),
                        torch.empty(1, device=DEV), ws)
    with pytest.raises(twa.TwaError):
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_SLAB_ROWS, 65536 + 512)
    torch.cuda.synchronize()
    twa.twa_destroy(ctx)
    twa.twa_destroy(ref)
