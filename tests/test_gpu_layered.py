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
    """Code values from the canonical image, by the oracle's definition of that image."""
    return orc.unpack_unsigned(packed.astype(np.uint8), D, bits)


ALL_BITS = [8, 4, 3, 2, 1, 16]              # the widths of the paper's bits ablation


def skip_unless_fits(bits, n):
    if bits == 16 and n > 64:
        pytest.skip("16-bit codes are stored as two 8-bit planes: n <= 64")


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


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("D,n,layers", CASES)
def test_quantize_affine_bit_exact(env, D, n, layers, bits):
    ctx, _ = env
    skip_unless_fits(bits, n)
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
    assert codes_g.numel() == n * ((D * orc.SLOT_BITS[bits] + 7) // 8)


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("lo,span", [(-0.37, 1.0), (0.0123, 3.3e-3), (-96.7, 200.1), (0.0, 2.9e-37), (-5.0, 2.5e38)])
def test_quantize_affine_near_half_integers_matches_the_ieee_quotient(env, bits, lo, span):
    """Elements whose quotient (e - b) / a sits on, or within a few ulps of, a half-integer, where the
    code hangs on the last bit of the IEEE float32 operations the oracle performs; two layers with
    different factors, one of them with a tiny or huge scale."""
    ctx, _ = env
    top = 2 ** bits - 1
    cols = []
    for lo_l, span_l in ((lo, span), (0.25, 0.731)):
        lo32 = np.float32(lo_l)
        hi32 = np.float32(np.float64(lo32) + span_l)
        a32 = np.float32(hi32 - lo32) / np.float32(top)
        ks = np.arange(0, min(top, 300), dtype=np.float64) + 0.5
        with np.errstate(over="ignore", under="ignore"):
            base = (np.float64(lo32) + ks * np.float64(a32)).astype(np.float32)
            vals = [base]
            for _ in range(5):
                vals.append(np.nextafter(vals[-1], np.float32(np.inf)))
            dn = base
            for _ in range(5):
                dn = np.nextafter(dn, np.float32(-np.inf))
                vals.append(dn)
        col = np.concatenate(vals + [np.array([lo32, hi32], dtype=np.float32)])
        cols.append(np.clip(col, lo32, hi32))
    layers = [0, cols[0].size, cols[0].size + cols[1].size]
    D = layers[-1]
    n = 2
    P = torch.zeros((n, inputs.padded_ld(D, 4)), dtype=torch.float32, device=DEV)
    flat = np.concatenate(cols)
    P[0, :D] = torch.from_numpy(flat).to(DEV)
    P[1, :D] = torch.from_numpy(np.concatenate([c[::-1] for c in cols])).to(DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    lb = twa.twa_quantize_affine(ctx, twa.basis_from_tensor(P, D), layers, bits, lws)
    status_ok(ctx)
    codes_g, a_g, b_g = twa.twa_layered_export(ctx, lb)
    codes_o, a_o, b_o = orc.affine_quantize(np.asfortranarray(P[:, :D].cpu().numpy().T), layers, bits)
    np.testing.assert_array_equal(a_g.cpu().numpy(), a_o)
    np.testing.assert_array_equal(b_g.cpu().numpy(), b_o)
    np.testing.assert_array_equal(unpack_unsigned(codes_g.cpu().numpy(), D, bits), codes_o)


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("D,n,layers,chunk_rows", [
    (1777, 6, [0, 7, 300, 301, 1000, 1777], 500),              # chunk edges inside layers and inside 16-byte code groups
    (70001, 33, [0, 64, 1000, 1001, 30000, 30017, 65536, 70001], 8192),
    (70001, 33, [0, 64, 1000, 1001, 30000, 30017, 65536, 70001], 70004),   # one chunk
    (300000, 20, [0, 300000], 65536),
    (5, 2, [0, 1, 5], 4),
])
def test_chunked_layered_build_matches_oracle_and_resident_build(env, D, n, layers, chunk_rows, bits):
    """The row-chunked build gives the mean bit for bit, float32 vectors equal to the resident build's
    up to the last bit (the norms are summed in another grouping), and codes and factors that are
    exactly the oracle's quantiser applied to the float32 vectors of its own pass 1."""
    skip_unless_fits(bits, n)
    ctx, _ = env
    ld = inputs.padded_ld(D, 4)
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 43, DEV, ld=ld)
    A = W[:, :D].cpu().numpy().T.copy()
    lws = twa.new_layered_workspace(layers, n, DEV)
    wbar = torch.full((D + 3,), 7.0, device=DEV)[:D]
    lb = twa.twa_layered_build_begin(ctx, D, n, layers, bits, lws, DEV)
    Q = torch.zeros((n, ld), device=DEV)
    # the second pass runs over another chunking: the result may not depend on it
    sizes = [chunk_rows, max(4, (chunk_rows // 3) // 4 * 4), chunk_rows]
    for p in range(3):
        for r0 in range(0, D, sizes[p]):
            rows = min(sizes[p], D - r0)
            chunk = W[:, r0:r0 + rows]                    # a view: column stride ld, 16-byte aligned start
            twa.twa_layered_build_feed(ctx, lb, p, chunk, r0, rows, wbar, lws,
                                       q32_out=Q[:, r0:r0 + rows] if p == 1 else None)
        twa.twa_layered_build_end_pass(ctx, lb, p, lws)
    status_ok(ctx)
    P_o, wbar_o = orc.center_normalize(A, layers)
    np.testing.assert_array_equal(wbar.cpu().numpy(), wbar_o.astype(np.float32))
    Qg = np.asfortranarray(Q[:, :D].cpu().numpy().T)
    # against the resident build on the same candidates
    W2 = W.clone()
    wbar2 = torch.empty(D, device=DEV)
    twa.twa_build_centered(ctx, W2, D, layers, wbar2, lws)
    Pr = W2[:, :D].cpu().numpy().T
    assert np.max(np.abs(Qg - Pr)) <= 2 * np.finfo(np.float32).eps * max(1e-30, np.max(np.abs(Pr)))
    scale = np.abs(A).max()
    for l in range(len(layers) - 1):
        r0, r1 = layers[l], layers[l + 1]
        norms = np.linalg.norm(A[r0:r1].astype(np.float64) - wbar_o[r0:r1, None], axis=0)
        tol = 4 * np.finfo(np.float32).eps * np.maximum(1.0, scale * np.sqrt(r1 - r0) / np.maximum(norms, 1e-300))
        assert np.all(np.abs(Qg[r0:r1] - P_o[r0:r1]).max(axis=0) <= tol)
    codes_g, a_g, b_g = twa.twa_layered_export(ctx, lb)
    codes_o, a_o, b_o = orc.affine_quantize(Qg, layers, bits)
    np.testing.assert_array_equal(a_g.cpu().numpy(), a_o)
    np.testing.assert_array_equal(b_g.cpu().numpy(), b_o)
    np.testing.assert_array_equal(unpack_unsigned(codes_g.cpu().numpy(), D, bits), codes_o)
    # the basis steps like any other layered basis
    sws = twa.new_layered_step_workspace(lb)
    L = len(layers) - 1
    gen = torch.Generator(device=DEV)
    gen.manual_seed(D + n)
    g = torch.randn(D, generator=gen, device=DEV) * 1e-3
    c = torch.empty((L, n), device=DEV)
    twa.twa_layered_project(ctx, lb, g, c, sws)
    status_ok(ctx)
    c_o = orc.project_layerwise(codes_o, layers, a_o, b_o, g.cpu().numpy())
    scale_c = _term_scale(codes_o, layers, a_o, b_o, g.double().cpu().numpy())
    assert np.all(np.abs(c.cpu().numpy() - c_o) <= 1e-5 * np.maximum(scale_c, 1e-30))


def test_chunked_layered_build_rejects_bad_arguments(env):
    ctx, _ = env
    D, n, layers = 5000, 3, [0, 100, 5000]
    lws = twa.new_layered_workspace(layers, n, DEV)
    lb = twa.twa_layered_build_begin(ctx, D, n, layers, 8, lws, DEV)
    chunk = torch.zeros((n, 1024), device=DEV)
    wbar = torch.empty(D, device=DEV)
    with pytest.raises(twa.TwaError) as e:
        twa.twa_layered_build_feed(ctx, lb, 0, chunk, 4990, 1024, wbar, lws)       # past the end
    assert e.value.code == twa.TWA_ERR_INVALID_ARG
    with pytest.raises(twa.TwaError) as e:
        twa.twa_layered_build_feed(ctx, lb, 0, chunk, 1022, 1024, wbar, lws)       # row0 not a multiple of 4
    assert e.value.code == twa.TWA_ERR_MISALIGNED
    with pytest.raises(twa.TwaError) as e:
        twa.twa_layered_build_feed(ctx, lb, 3, chunk, 0, 1024, wbar, lws)          # no such pass
    assert e.value.code == twa.TWA_ERR_INVALID_ARG
    status_ok(ctx)


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


# ------------------------------------------------------------------ layer-wise step
def _random_layers(D, count, seed):
    rng = np.random.default_rng(seed)
    cuts = np.unique(rng.integers(1, D, size=count - 1))
    return [0] + [int(x) for x in cuts] + [D]


STEP_CASES = CASES + [
    (3_000_017, 33, _random_layers(3_000_017, 60, 1)),        # two 512-byte segments per tile column
    (2_500_003, 100, _random_layers(2_500_003, 40, 2)),       # one segment per tile column
    (1_200_000, 128, [0, 5, 6, 70, 1_200_000]),
]


def _layered_basis(ctx, D, n, layers, bits, seed):
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, seed, DEV, ld=inputs.padded_ld(D, 4))
    wbar = torch.empty(D, device=DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
    lb = twa.twa_quantize_affine(ctx, P32, layers, bits, lws)
    codes_g, a_g, b_g = twa.twa_layered_export(ctx, lb)
    status_ok(ctx)
    codes = unpack_unsigned(codes_g.cpu().numpy(), D, bits)
    return lb, wbar, codes, a_g.cpu().numpy(), b_g.cpu().numpy()


def _term_scale(codes, layers, a, b, g64):
    """Per (layer, column) sum of the magnitudes of the terms of c: the size rounding errors scale with."""
    L, n = len(layers) - 1, codes.shape[1]
    s = np.zeros((L, n))
    ag = np.abs(g64)
    for l in range(L):
        r0, r1 = layers[l], layers[l + 1]
        s[l] = abs(float(a[l])) * (codes[r0:r1].astype(np.float64).T @ ag[r0:r1]) + abs(float(b[l])) * ag[r0:r1].sum()
    return s


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("D,n,layers", STEP_CASES)
def test_layered_project(env, D, n, layers, bits, g_dtype):
    ctx, _ = env
    skip_unless_fits(bits, n)
    lb, _, codes, a, b = _layered_basis(ctx, D, n, layers, bits, 51)
    L = len(layers) - 1
    g = inputs.gradient(D, 1e-3, 7, 0, g_dtype, DEV)
    sws = twa.new_layered_step_workspace(lb)
    c = torch.full((L, n), float("nan"), device=DEV)
    twa.twa_layered_project(ctx, lb, g, c, sws)
    status_ok(ctx)
    g64 = g.float().cpu().numpy().astype(np.float64)
    c_o = orc.project_layerwise(codes, layers, a, b, g64)
    c_g = c.cpu().numpy()
    assert rel(c_g, c_o) <= TOL
    assert np.all(np.abs(c_g - c_o) <= 2e-6 * _term_scale(codes, layers, a, b, g64) + 1e-30)
    # same call again: bitwise the same result (fixed summation order)
    c2 = torch.empty_like(c)
    twa.twa_layered_project(ctx, lb, g, c2, sws)
    assert torch.equal(c, c2)


@pytest.mark.parametrize("with_base", [True, False])
@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("D,n,layers", STEP_CASES)
def test_layered_lift(env, D, n, layers, bits, with_base):
    ctx, _ = env
    skip_unless_fits(bits, n)
    lb, wbar, codes, a, b = _layered_basis(ctx, D, n, layers, bits, 52)
    L = len(layers) - 1
    gen = torch.Generator(device="cpu").manual_seed(5)
    beta = (torch.randn((L, n), generator=gen) * 0.3).to(DEV)
    if L > 2:
        beta[1] = 0.0                                          # a layer that stays at its mean
    sws = twa.new_layered_step_workspace(lb)
    w = torch.full((D,), float("nan"), device=DEV)
    twa.twa_layered_lift(ctx, lb, beta, wbar if with_base else None, w, sws)
    status_ok(ctx)
    base = wbar.cpu().numpy() if with_base else None
    w_o = orc.lift_layerwise(codes, layers, a, b, beta.cpu().numpy(), base)
    w_g = w.cpu().numpy()
    assert rel(w_g, w_o) <= TOL
    d_o = w_o - (base.astype(np.float64) if with_base else 0.0)
    d_g = w_g.astype(np.float64) - (base.astype(np.float64) if with_base else 0.0)
    assert np.linalg.norm(d_g - d_o) <= (2e-5 if with_base else TOL) * np.linalg.norm(d_o)
    if L > 2 and with_base:
        r0, r1 = layers[1], layers[2]
        np.testing.assert_array_equal(w_g[r0:r1], base[r0:r1])


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("D,n,layers", STEP_CASES[1:2] + STEP_CASES[4:6])
def test_layered_step_matches_oracle_over_iterations(env, D, n, layers, bits):
    ctx, _ = env
    skip_unless_fits(bits, n)
    lb, wbar, codes, a, b = _layered_basis(ctx, D, n, layers, bits, 53)
    L = len(layers) - 1
    sws = twa.new_layered_step_workspace(lb)
    beta = torch.zeros((L, n), device=DEV)
    w = torch.empty(D, device=DEV)
    c = torch.empty((L, n), device=DEV)
    beta_o = np.zeros((L, n))
    wbar_o = wbar.cpu().numpy()
    lr, lam = 0.5, 1e-2
    for it in range(3):
        g = inputs.gradient(D, 1e-2, 9, it, torch.bfloat16, DEV)
        twa.twa_layered_step(ctx, lb, g, lr, lam, beta, wbar, w, sws, c_out=c)
        status_ok(ctx)
        # the oracle continues from the GPU's float32 coefficients, so errors do not compound
        beta_new_o, w_o, c_o = orc.step_layerwise(codes, layers, a, b, g.float().cpu().numpy(), beta_o, wbar_o,
                                                  lr, lam)
        assert rel(c.cpu().numpy(), c_o) <= TOL
        assert rel(beta.cpu().numpy(), beta_new_o) <= TOL
        w_from_gpu_beta = orc.lift_layerwise(codes, layers, a, b, beta.cpu().numpy(), wbar_o)
        assert rel(w.cpu().numpy(), w_from_gpu_beta) <= TOL
        assert rel(w.cpu().numpy(), w_o) <= 2e-5
        beta_o = beta.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("bits", [8, 4])
def test_groups_of_layers_as_separate_bases_step_like_the_whole(env, bits):
    """Layers do not interact (Section 4.5), so a model may be held as several layered bases over
    consecutive groups of layers -- the way a model of more than 2^31 rows is held: the same factors and
    codes as the one basis over all layers, and after three steps the same coefficients and weights
    (to rounding: the layers sit differently in the kernels' tiles), both within the bound of the oracle
    on the whole model."""
    ctx, _ = env
    D, n, layers = 90001, 12, [0, 100, 101, 30000, 65536, 90001]
    cut_layer, cut = 3, 30000
    L = len(layers) - 1
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 61, DEV, ld=inputs.padded_ld(D, 4))
    parts = []
    for r0, r1, ls in ((0, cut, layers[:cut_layer + 1]), (cut, D, [o - cut for o in layers[cut_layer:]])):
        Wp = torch.zeros((n, inputs.padded_ld(r1 - r0, 4)), device=DEV)
        Wp[:, :r1 - r0] = W[:, r0:r1]
        wbar_p = torch.empty(r1 - r0, device=DEV)
        lws = twa.new_layered_workspace(ls, n, DEV)
        lb_p = twa.twa_quantize_affine(ctx, twa.twa_build_centered(ctx, Wp, r1 - r0, ls, wbar_p, lws), ls, bits, lws)
        parts.append((r0, r1, ls, lb_p, wbar_p, twa.new_layered_step_workspace(lb_p), Wp))
    wbar = torch.empty(D, device=DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    lb = twa.twa_quantize_affine(ctx, twa.twa_build_centered(ctx, W, D, layers, wbar, lws), layers, bits, lws)
    codes_g, a_g, b_g = twa.twa_layered_export(ctx, lb)
    status_ok(ctx)
    l0 = 0
    for r0, r1, ls, lb_p, wbar_p, _, _ in parts:
        cp, ap, bp = twa.twa_layered_export(ctx, lb_p)
        Lp = len(ls) - 1
        assert torch.equal(ap, a_g[l0:l0 + Lp]) and torch.equal(bp, b_g[l0:l0 + Lp])
        np.testing.assert_array_equal(unpack_unsigned(cp.cpu().numpy(), r1 - r0, bits),
                                      unpack_unsigned(codes_g.cpu().numpy(), D, bits)[r0:r1])
        assert torch.equal(wbar_p, wbar[r0:r1])
        l0 += Lp
    codes = unpack_unsigned(codes_g.cpu().numpy(), D, bits)
    a, b = a_g.cpu().numpy(), b_g.cpu().numpy()
    sws = twa.new_layered_step_workspace(lb)
    beta, w = torch.zeros((L, n), device=DEV), torch.empty(D, device=DEV)
    beta_p, w_p = torch.zeros((L, n), device=DEV), torch.empty(D, device=DEV)
    beta_o, wbar_o = np.zeros((L, n)), wbar.cpu().numpy()
    lr, lam = 0.5, 1e-2
    for it in range(3):
        g = inputs.gradient(D, 1e-2, 10, it, torch.bfloat16, DEV)
        twa.twa_layered_step(ctx, lb, g, lr, lam, beta, wbar, w, sws)
        l0 = 0
        for r0, r1, ls, lb_p, wbar_p, sws_p, _ in parts:
            Lp = len(ls) - 1
            twa.twa_layered_step(ctx, lb_p, g[r0:r1], lr, lam, beta_p[l0:l0 + Lp], wbar_p, w_p[r0:r1], sws_p)
            l0 += Lp
        status_ok(ctx)
        beta_o, w_o, _ = orc.step_layerwise(codes, layers, a, b, g.float().cpu().numpy(), beta_o, wbar_o, lr, lam)
        assert rel(beta_p.cpu().numpy(), beta.cpu().numpy()) <= 1e-6
        assert rel(beta_p.cpu().numpy(), beta_o) <= TOL and rel(beta.cpu().numpy(), beta_o) <= TOL
        assert rel(w_p.cpu().numpy(), w_o) <= 2e-5
        assert torch.max(torch.abs(w_p - w)).item() <= 4 * np.spacing(np.float32(np.abs(w_o).max()))


@pytest.mark.parametrize("bits", [8, 4])
def test_layered_step_replayed_from_a_cuda_graph(bits):
    """twa_layered_step (three launches) captured once and replayed on new gradient bytes: the same
    coefficients and weights as direct calls, bit for bit."""
    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    D, n, layers = 90001, 12, [0, 100, 101, 30000, 65536, 90001]
    L = len(layers) - 1
    with torch.cuda.stream(stream):
        ctx = twa.twa_create(0, stream=stream)
        lb, wbar, _, _, _ = _layered_basis(ctx, D, n, layers, bits, 77)
        sws = twa.new_layered_step_workspace(lb)
        gs = [inputs.gradient(D, 1e-2, 3, it, torch.bfloat16, DEV) for it in range(6)]
        beta_d, w_d = torch.zeros((L, n), device=DEV), torch.empty(D, device=DEV)
        for g in gs:
            twa.twa_layered_step(ctx, lb, g, 0.5, 1e-2, beta_d, wbar, w_d, sws)
        g_buf = torch.zeros(D, device=DEV, dtype=torch.bfloat16)
        beta_g, w_g = torch.zeros((L, n), device=DEV), torch.empty(D, device=DEV)
        twa.twa_layered_step(ctx, lb, g_buf, 0.5, 1e-2, beta_g, wbar, w_g, sws)     # warm-up outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            twa.twa_layered_step(ctx, lb, g_buf, 0.5, 1e-2, beta_g, wbar, w_g, sws)
        beta_g.zero_()
        for g in gs:
            g_buf.copy_(g)
            graph.replay()
        stream.synchronize()
        status_ok(ctx)
        assert torch.equal(beta_g, beta_d) and torch.equal(w_g, w_d)
        del graph
        twa.twa_destroy(ctx)


def test_layered_step_reports_nonfinite_and_bad_arguments(env):
    ctx, _ = env
    D, n, layers = 40000, 5, [0, 100, 20000, 40000]
    lb, wbar, _, _, _ = _layered_basis(ctx, D, n, layers, 8, 54)
    sws = twa.new_layered_step_workspace(lb)
    g = inputs.gradient(D, 1e-3, 7, 0, torch.float32, DEV)
    g[30000] = float("inf")
    c = torch.empty((3, n), device=DEV)
    twa.twa_layered_project(ctx, lb, g, c, sws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_NONFINITE, 2)
    twa.twa_clear_status(ctx)
    assert torch.isfinite(c[:2]).all() and torch.isnan(c[2]).all()
    beta = torch.zeros((3, n), device=DEV)
    beta[1, 2] = float("nan")
    w = torch.empty(D, device=DEV)
    twa.twa_layered_lift(ctx, lb, beta, wbar, w, sws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_NONFINITE, 1)
    twa.twa_clear_status(ctx)
    assert torch.isnan(w[100:20000]).all() and torch.isfinite(w[:100]).all() and torch.isfinite(w[20000:]).all()
    with pytest.raises(twa.TwaError) as e:
        twa.twa_layered_project(ctx, lb, g, c, sws[: sws.numel() - 256])
    assert e.value.code == twa.TWA_ERR_WORKSPACE
