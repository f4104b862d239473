"""GPU parity: every C-ABI call against the float64 CPU oracle on the same seeded bytes.

Sizes span several tiles (a tile is 512 rows at 8 bits, 1024 at 4 bits, 128 at 32 bits),
ragged tails (D not a multiple of 2, 4, 16, 128) and the column counts 1, 2, 3, 33, 100, 128.
Bounds: codes and scales bit-exact; projection, lift and step within 1e-5 relative L2;
basis orthonormal to 1e-5.
"""

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


def rel(x, y):
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    d = np.linalg.norm(y)
    return np.linalg.norm(x - y) / d if d > 0 else np.linalg.norm(x)


def status_ok(ctx):
    code, detail = twa.twa_get_status(ctx)
    assert code == 0, (twa.twa_strerror(code), detail)


def random_basis(D, n, seed, scale=1.0):
    """float32 matrix (n, ld) on the GPU with unit-ish columns of different magnitude."""
    ld = inputs.padded_ld(D, 4)
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    P = torch.zeros((n, ld), dtype=torch.float32, device=DEV)
    P[:, :D] = torch.randn((n, D), generator=g, device=DEV) * scale / np.sqrt(D)
    P[:, :D] *= (1.0 + torch.arange(n, device=DEV, dtype=torch.float32))[:, None] * 0.37
    return P


def host_cols(P, D):
    return P[:, :D].cpu().numpy().T          # (D, n) view with contiguous columns


SHAPES = [(1, 1), (5, 2), (127, 3), (513, 1), (1024, 2), (4099, 33), (70001, 100), (33333, 128),
          (300007, 20)]


# ------------------------------------------------------------------ mean
@pytest.mark.parametrize("D,n", [(1, 1), (6, 3), (1023, 7), (40002, 33)])
def test_mean(env, D, n):
    ctx, _ = env
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 3, DEV, ld=inputs.padded_ld(D, 4))
    wbar = torch.full((D + 8,), 7.0, dtype=torch.float32, device=DEV)
    twa.twa_mean(ctx, W, D, wbar)
    status_ok(ctx)
    ref = orc.mean(host_cols(W, D)).astype(np.float32)
    np.testing.assert_array_equal(wbar[:D].cpu().numpy(), ref)
    assert torch.all(wbar[D:] == 7.0)            # nothing written past D


# ------------------------------------------------------------------ quantiser
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("D,n", SHAPES)
def test_quantize_bit_exact(env, D, n, bits):
    ctx, ws = env
    P = random_basis(D, n, 11 + D)
    if n >= 3:
        P[1].zero_()                              # an all-zero column
        P[2, :D] = -P[2, :D].abs()                # absmax element negative
    P32 = twa.basis_from_tensor(P, D)
    Pq = twa.twa_quantize_basis(ctx, P32, bits, ws)
    status_ok(ctx)
    codes_g, s_g = twa.twa_basis_export(ctx, Pq)
    codes_o, s_o = orc.quantize(np.asfortranarray(host_cols(P, D)), bits)
    np.testing.assert_array_equal(s_g.cpu().numpy(), s_o)
    np.testing.assert_array_equal(codes_g.cpu().numpy(), orc.pack_codes(codes_o, bits))
    assert Pq.data.numel() == twa.twa_basis_bytes(D, n, bits)
    assert codes_g.numel() + 4 * n == orc.storage_bytes(D, n, bits)


def test_quantize_ties_round_to_even(env):
    ctx, ws = env
    vals = [127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, -126.5, 64.5]
    P = torch.zeros((2, 12), dtype=torch.float32, device=DEV)
    P[0, :10] = torch.tensor(vals, device=DEV)
    P[1, :10] = torch.tensor([7.0, 0.5, 1.5, 2.5, -3.5, -6.5, 6.5, -7.0, 4.5, 5.5], device=DEV)
    P32 = twa.basis_from_tensor(P, 10)
    for bits, row, want in ((8, 0, [127, 0, 2, 2, 0, -2, -2, 4, -126, 64]),
                            (4, 1, [7, 0, 2, 2, -4, -6, 6, -7, 4, 6])):
        Pq = twa.twa_quantize_basis(ctx, P32, bits, ws)
        codes, s = twa.twa_basis_export(ctx, Pq)
        got = orc.unpack_codes(codes.cpu().numpy(), 10, bits)
        assert s[row].item() == 1.0
        np.testing.assert_array_equal(got[:, row], want)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("absmax", [1.0, 0.0123, 3.3e-3, 96.7, 2.9e-37, 1.1e-44, 2.5e38])
def test_quantize_near_half_integers_matches_the_ieee_quotient(env, bits, absmax):
    """Elements whose quotient p / s sits on, or within a few ulps of, a half-integer: the code then
    hangs on the last bit of the IEEE float32 quotient (what the oracle rounds), for scales that are
    not powers of two, for a scale so small that it is subnormal, and for a huge one."""
    ctx, ws = env
    qmax = 127 if bits == 8 else 7
    am = np.float32(absmax)
    sc = np.float32(am) / np.float32(qmax)
    ks = np.arange(-qmax, qmax, dtype=np.float64) + 0.5
    with np.errstate(over="ignore", under="ignore"):
        base = (ks * np.float64(sc)).astype(np.float32)
        vals = [base]
        for _ in range(6):
            vals.append(np.nextafter(vals[-1], np.float32(np.inf)))
        lo = base
        for _ in range(6):
            lo = np.nextafter(lo, np.float32(-np.inf))
            vals.append(lo)
    col = np.concatenate(vals + [np.array([am, -am, 0.0], dtype=np.float32)])
    col = col[np.abs(col) <= am]
    D = col.size
    P = torch.zeros((2, inputs.padded_ld(D, 4)), dtype=torch.float32, device=DEV)
    P[0, :D] = torch.from_numpy(col).to(DEV)
    P[1, :D] = torch.from_numpy(col[::-1].copy()).to(DEV)
    Pq = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), bits, ws)
    status_ok(ctx)
    codes_g, s_g = twa.twa_basis_export(ctx, Pq)
    codes_o, s_o = orc.quantize(np.asfortranarray(host_cols(P, D)), bits)
    assert s_o[0] == sc
    np.testing.assert_array_equal(s_g.cpu().numpy(), s_o)
    np.testing.assert_array_equal(codes_g.cpu().numpy(), orc.pack_codes(codes_o, bits))
    # the case is what it claims: many of these quotients round differently from their neighbours one ulp away
    if sc > 1e-40:
        c = codes_o[: base.size * 13, 0].reshape(13, base.size)
        assert np.count_nonzero(c.max(axis=0) != c.min(axis=0)) >= base.size // 2


@pytest.mark.parametrize("bits", [8, 4])
def test_export_import_roundtrip(env, bits):
    ctx, ws = env
    D, n = 7001, 5
    P = random_basis(D, n, 5)
    Pq = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), bits, ws)
    codes, s = twa.twa_basis_export(ctx, Pq)
    Pq2 = twa.twa_basis_import(ctx, codes, s, D, bits)
    codes2, s2 = twa.twa_basis_export(ctx, Pq2)
    status_ok(ctx)
    assert torch.equal(codes, codes2) and torch.equal(s, s2)
    g = torch.randn(D, device=DEV)
    c1 = torch.empty(n, device=DEV)
    c2 = torch.empty(n, device=DEV)
    twa.twa_project(ctx, Pq, g, c1, ws)
    twa.twa_project(ctx, Pq2, g, c2, ws)
    assert torch.equal(c1, c2)


# ------------------------------------------------------------------ project / lift
@pytest.fixture(params=[0, 1], ids=["tensor-pipe", "float-fma"])
def dequant_path(request, env):
    """Both ways the library turns 8/4-bit codes into products (TWA_TUNE_DEQUANT_PATH)."""
    ctx, _ = env
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_DEQUANT_PATH, request.param)
    yield request.param
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_DEQUANT_PATH, 0)


@pytest.mark.parametrize("gdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bits", [32, 8, 4])
@pytest.mark.parametrize("D,n", SHAPES)
def test_project_and_lift(env, dequant_path, D, n, bits, gdt):
    ctx, ws = env
    if bits == 32 and dequant_path == 1:
        pytest.skip("the path choice only exists for 8/4-bit storage")
    P = random_basis(D, n, 100 + D + n)
    P32 = twa.basis_from_tensor(P, D)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(D * 7 + n)
    g = (torch.randn(D + 16, generator=gen, device=DEV) * 1e-3).to(gdt)
    g[D:] = float("nan")                           # must never be read
    alpha = torch.randn(n, generator=gen, device=DEV)
    base = torch.randn(D, generator=gen, device=DEV)
    if bits == 32:
        B = P32
        Ph = host_cols(P, D)
        proj = lambda gg: orc.project_f32(Ph, gg)
        lift = lambda a, b: orc.lift_f32(Ph, a, b)
    else:
        B = twa.twa_quantize_basis(ctx, P32, bits, ws)
        codes, s = twa.twa_basis_export(ctx, B)
        co = orc.unpack_codes(codes.cpu().numpy(), D, bits)
        so = s.cpu().numpy()
        proj = lambda gg: orc.project(co, so, gg)
        lift = lambda a, b: orc.lift(co, so, a, b)
    c = torch.full((n + 4,), 3.0, device=DEV)
    twa.twa_project(ctx, B, g[:D], c, ws)
    status_ok(ctx)
    c_ref = proj(g[:D].float().cpu().numpy())
    assert rel(c[:n].cpu().numpy(), c_ref) <= TOL
    assert torch.all(c[n:] == 3.0)

    w = torch.full((D + 8,), 5.0, device=DEV)
    twa.twa_lift(ctx, B, alpha, None, w, ws)       # P alpha alone: the meaningful bound
    status_ok(ctx)
    assert rel(w[:D].cpu().numpy(), lift(alpha.cpu().numpy(), None)) <= TOL
    assert torch.all(w[D:] == 5.0)
    twa.twa_lift(ctx, B, alpha, base, w, ws)
    w_ref = lift(alpha.cpu().numpy(), base.cpu().numpy())
    assert rel(w[:D].cpu().numpy(), w_ref) <= TOL
    assert np.max(np.abs(w[:D].cpu().numpy() - w_ref.astype(np.float32))) <= 4 * np.spacing(
        np.float32(np.max(np.abs(w_ref))))
    # in place: base and output the same buffer
    w2 = base.clone()
    twa.twa_lift(ctx, B, alpha, w2, w2, ws)
    assert torch.equal(w2, w[:D])


@pytest.mark.parametrize("bits", [32, 8, 4])
def test_step_sequence_and_determinism(env, dequant_path, bits):
    ctx, ws = env
    if bits == 32 and dequant_path == 1:
        pytest.skip("the path choice only exists for 8/4-bit storage")
    D, n, lr, lam = 50021, 24, 0.1, 0.05
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 9, DEV, ld=inputs.padded_ld(D, 4))
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    B = P32 if bits == 32 else twa.twa_quantize_basis(ctx, P32, bits, ws)
    if bits == 32:
        Ph = host_cols(W, D)
        ostep = lambda g, a: orc.step_f32(Ph, g, a, wbar.cpu().numpy(), lr, lam)
    else:
        codes, s = twa.twa_basis_export(ctx, B)
        co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
        ostep = lambda g, a: orc.step(co, so, g, a, wbar.cpu().numpy(), lr, lam)
    runs = []
    for rep in range(2):
        alpha = torch.zeros(n, device=DEV)
        w = torch.empty(D, device=DEV)
        c = torch.empty(n, device=DEV)
        a_o = np.zeros(n)
        outs = []
        for t in range(4):
            g = inputs.gradient(D, 1e-3, 9, t, torch.float32, DEV)
            twa.twa_step(ctx, B, g, lr, lam, alpha, wbar, w, ws, c_out=c)
            status_ok(ctx)
            if rep == 0:
                a_o, w_o, c_o = ostep(g.cpu().numpy(), a_o)
                assert rel(c.cpu().numpy(), c_o) <= TOL
                assert rel(alpha.cpu().numpy(), a_o) <= TOL
                assert rel(w.cpu().numpy(), w_o) <= TOL
                assert rel(w.cpu().numpy().astype(np.float64) - wbar.cpu().numpy(),
                           w_o - wbar.cpu().numpy()) <= 1e-3   # increment, carried by a float32 w
            outs.append((alpha.clone(), w.clone(), c.clone()))
        runs.append(outs)
    for (a1, w1, c1), (a2, w2, c2) in zip(*runs):
        assert torch.equal(a1, a2) and torch.equal(w1, w2) and torch.equal(c1, c2)


@pytest.mark.parametrize("bits,gdt", [(8, torch.bfloat16), (4, torch.float32), (32, torch.float32)])
def test_step_replayed_from_a_cuda_graph(bits, gdt):
    """A training loop may capture twa_step once and replay it: the call only enqueues kernels (tensor
    maps and arguments are fixed at capture), so a replay with new bytes in the same gradient buffer
    is the next step.  Ten replayed steps against ten direct calls (bit for bit) and against the oracle."""
    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    D, n, steps = 150001, 24, 10
    with torch.cuda.stream(stream):
        ctx = twa.twa_create(0, stream=stream)
        ws = twa.new_workspace(DEV)
        P = random_basis(D, n, 808)
        B = twa.basis_from_tensor(P, D)
        if bits != 32:
            B = twa.twa_quantize_basis(ctx, B, bits, ws)
            codes, s = twa.twa_basis_export(ctx, B)
            co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
        gen = torch.Generator(device=DEV)
        gen.manual_seed(99)
        gs = [(torch.randn(D, generator=gen, device=DEV) * 1e-3).to(gdt) for _ in range(steps)]
        wbar = torch.randn(D, generator=gen, device=DEV)
        # direct calls
        alpha_d = torch.zeros(n, device=DEV)
        w_d = torch.empty(D, device=DEV)
        for g in gs:
            twa.twa_step(ctx, B, g, 0.1, 0.01, alpha_d, wbar, w_d, ws)
        # one captured call, replayed on fresh bytes in the same buffers
        g_buf = torch.zeros(D, device=DEV, dtype=gdt)
        alpha_g = torch.zeros(n, device=DEV)
        w_g = torch.empty(D, device=DEV)
        twa.twa_step(ctx, B, g_buf, 0.1, 0.01, alpha_g, wbar, w_g, ws)      # warm-up outside the capture
        alpha_g.zero_()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            twa.twa_step(ctx, B, g_buf, 0.1, 0.01, alpha_g, wbar, w_g, ws)
        alpha_g.zero_()
        for g in gs:
            g_buf.copy_(g)
            graph.replay()
        stream.synchronize()
        status_ok(ctx)
        assert torch.equal(alpha_g, alpha_d) and torch.equal(w_g, w_d)
        a_o = np.zeros(n)
        for g in gs:
            g_h = g.float().cpu().numpy()
            if bits != 32:
                a_o, w_o, _ = orc.step(co, so, g_h, a_o, wbar.cpu().numpy(), 0.1, 0.01)
            else:
                a_o, w_o, _ = orc.step_f32(host_cols(P, D), g_h, a_o, wbar.cpu().numpy(), 0.1, 0.01)
        assert rel(alpha_g.cpu().numpy(), a_o) <= TOL
        assert rel(w_g.cpu().numpy(), w_o) <= TOL
        del graph
        twa.twa_destroy(ctx)


def test_step_host_matches_device_step(env):
    ctx, ws = env
    D, n = 30011, 10
    P = random_basis(D, n, 77)
    B = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), 8, ws)
    wbar = torch.randn(D, device=DEV)
    g = (torch.randn(D, device=DEV) * 1e-3).bfloat16()
    a1 = torch.zeros(n, device=DEV)
    a2 = torch.zeros(n, device=DEV)
    w1 = torch.empty(D, device=DEV)
    w2 = torch.empty(D, device=DEV)
    twa.twa_step(ctx, B, g, 0.1, 0.0, a1, wbar, w1, ws)
    g_host = g.cpu().pin_memory()
    w_host = torch.empty(D, dtype=torch.float32).pin_memory()
    g_stage = torch.empty(D, dtype=torch.bfloat16, device=DEV)
    twa.twa_step_host(ctx, B, g_host, 0.1, 0.0, a2, wbar, w2, w_host, g_stage, ws)
    status_ok(ctx)
    assert torch.equal(a1, a2) and torch.equal(w1, w2) and torch.equal(w_host, w1.cpu())


@pytest.mark.parametrize("bits,gdt", [(8, torch.bfloat16), (4, torch.float32), (32, torch.float32)])
def test_step_host_in_row_chunks_matches_device_step_and_oracle(env, bits, gdt):
    """From 2^22 rows on twa_step_host cuts the step into row chunks that overlap with the host copies
    (a second stream, events): the coefficients are the sum of the chunks' projections, so they agree
    with twa_step within rounding, w with the oracle's lift of those coefficients; two calls in a row
    reuse the staging buffer and the events."""
    ctx, ws = env
    D, n = (1 << 22) + 70001, 5
    P = random_basis(D, n, 78)
    B = twa.basis_from_tensor(P, D)
    if bits != 32:
        B = twa.twa_quantize_basis(ctx, B, bits, ws)
        codes, s = twa.twa_basis_export(ctx, B)
        co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
    else:
        Ph = host_cols(P, D)
    wbar = torch.randn(D, device=DEV)
    a_dev = torch.zeros(n, device=DEV)
    a_host = torch.zeros(n, device=DEV)
    w_dev = torch.empty(D, device=DEV)
    w_stage = torch.empty(D, device=DEV)
    w_host = torch.empty(D, dtype=torch.float32).pin_memory()
    g_stage = torch.empty(D, dtype=gdt, device=DEV)
    a_o = np.zeros(n)
    for t in range(2):
        g = inputs.gradient(D, 1e-3, 5, t, gdt, DEV)
        g_pinned = g.cpu().pin_memory()
        twa.twa_step(ctx, B, g, 0.1, 0.0, a_dev, wbar, w_dev, ws)
        twa.twa_step_host(ctx, B, g_pinned, 0.1, 0.0, a_host, wbar, w_stage, w_host, g_stage, ws)
        status_ok(ctx)                                    # waits for the context's stream, hence for the copies
        gh = g.float().cpu().numpy()
        if bits != 32:
            a_o, w_o, _ = orc.step(co, so, gh, a_o, wbar.cpu().numpy(), 0.1)
        else:
            a_o, w_o, _ = orc.step_f32(Ph, gh, a_o, wbar.cpu().numpy(), 0.1)
        assert torch.equal(g_stage, g)
        assert rel(a_host.cpu().numpy(), a_o) <= TOL
        assert rel(a_host.cpu().numpy(), a_dev.cpu().numpy()) <= 1e-6
        assert torch.equal(w_host, w_stage.cpu())
        assert rel(w_host.numpy(), w_o) <= TOL
        assert np.max(np.abs(w_host.numpy() - w_o.astype(np.float32))) <= 4 * np.spacing(np.float32(np.abs(w_o).max()))


# ------------------------------------------------------------------ basis
@pytest.mark.parametrize("D,n", [(1, 1), (130, 2), (5003, 3), (70001, 33), (200004, 100), (40001, 128)])
def test_build_basis(env, D, n):
    ctx, ws = env
    if n > D:
        pytest.skip("n <= D required")
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 21, DEV, ld=inputs.padded_ld(D, 4))
    A = host_cols(W, D).copy()
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    status_ok(ctx)
    assert (P32.D, P32.n, P32.bits, P32.col_stride) == (D, n, 32, 4 * W.shape[1])
    np.testing.assert_array_equal(wbar.cpu().numpy(), orc.mean(A).astype(np.float32))
    Pg = host_cols(W, D).astype(np.float64)
    assert np.max(np.abs(Pg.T @ Pg - np.eye(n))) <= 1e-5
    Q, R, bad = orc.cgs2(A)
    assert bad is None
    # same factorisation: P^T A upper triangular with positive diagonal, A = P (P^T A)
    T = Pg.T @ A.astype(np.float64)
    assert np.all(np.diag(T) > 0)
    assert np.max(np.abs(np.tril(T, -1))) <= 2e-5 * np.max(np.abs(T))
    assert np.linalg.norm(A - Pg @ T) <= 1e-5 * np.linalg.norm(A)
    kappa = np.linalg.cond(A.astype(np.float64))
    assert np.max(np.linalg.norm(Pg - Q, axis=0)) <= 10 * kappa * np.finfo(np.float32).eps
    # pad columns untouched
    assert torch.all(W[:, D:] == 0)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("scale", [1e15, 1e-15])
def test_build_basis_on_very_large_and_very_small_candidates(env, scale, mode):
    """Q does not depend on the scale of the candidates: with columns of norm 1e15 and 1e-15 the build
    still returns the oracle's vectors (norms, Gram matrix and coefficients must not overflow or
    flush on the way)."""
    ctx, ws = env
    D, n = 60001, 19
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 5, DEV, ld=inputs.padded_ld(D, 4))
    W *= scale
    A = host_cols(W, D).copy()
    wbar = torch.empty(D, device=DEV)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, mode)
    try:
        twa.twa_build_basis(ctx, W, D, wbar, ws)
    finally:
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, 0)
    status_ok(ctx)
    Pg = host_cols(W, D).astype(np.float64)
    assert np.max(np.abs(Pg.T @ Pg - np.eye(n))) <= 1e-5
    Q, _, bad = orc.cgs2(A)
    assert bad is None
    kappa = np.linalg.cond(A.astype(np.float64))
    assert np.max(np.linalg.norm(Pg - Q, axis=0)) <= 10 * kappa * np.finfo(np.float32).eps
    np.testing.assert_array_equal(wbar.cpu().numpy(), orc.mean(A).astype(np.float32))


def test_basis_invariants_recover_candidates_and_reject_orthogonal(env):
    ctx, ws = env
    D, n = 60013, 10
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 0, DEV, ld=inputs.padded_ld(D, 4))
    A = W[:, :D].clone()
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    c = torch.empty(n, device=DEV)
    w = torch.empty(D, device=DEV)
    for i in range(n):
        twa.twa_project(ctx, P32, A[i].clone(), c, ws)
        twa.twa_lift(ctx, P32, c, None, w, ws)
        assert rel(w.cpu().numpy(), A[i].cpu().numpy()) <= 1e-5          # lift(project(w_i)) = w_i
        twa.twa_project(ctx, P32, A[i] - wbar, c, ws)
        twa.twa_lift(ctx, P32, c, wbar, w, ws)
        assert rel(w.cpu().numpy(), A[i].cpu().numpy()) <= 1e-5
    # alpha = 0 lifts to w_bar exactly
    twa.twa_lift(ctx, P32, torch.zeros(n, device=DEV), wbar, w, ws)
    assert torch.equal(w, wbar)
    # a vector orthogonal to the span (made so on the CPU in float64) projects to ~0
    A64 = A.cpu().numpy().T.astype(np.float64)
    x = np.random.default_rng(0).standard_normal(D)
    x -= A64 @ np.linalg.lstsq(A64, x, rcond=None)[0]
    xg = torch.tensor(x, dtype=torch.float32, device=DEV)
    twa.twa_project(ctx, P32, xg, c, ws)
    assert np.max(np.abs(c.cpu().numpy())) <= 1e-5 * np.linalg.norm(x)
    status_ok(ctx)


def test_rank_deficient_and_nonfinite_are_reported(env):
    ctx, ws = env
    D, n = 9001, 4
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 1, DEV, ld=inputs.padded_ld(D, 4))
    W[2] = W[0] * -2.0
    wbar = torch.empty(D, device=DEV)
    twa.twa_build_basis(ctx, W, D, wbar, ws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_RANK_DEFICIENT, 2)
    twa.twa_clear_status(ctx)
    status_ok(ctx)
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 1, DEV, ld=inputs.padded_ld(D, 4))
    W[1, 17] = float("inf")
    twa.twa_build_basis(ctx, W, D, wbar, ws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_NONFINITE, 1)
    twa.twa_clear_status(ctx)
    P = random_basis(D, n, 3)
    P[3, 5] = float("nan")
    twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), 8, ws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_NONFINITE, 3)
    twa.twa_clear_status(ctx)
    status_ok(ctx)


def test_host_side_argument_errors(env):
    ctx, ws = env
    D, n = 1000, 4
    P = random_basis(D, n, 1)
    P32 = twa.basis_from_tensor(P, D)
    g = torch.zeros(D + 4, device=DEV)
    c = torch.zeros(n, device=DEV)

    def code_of(fn):
        with pytest.raises(twa.TwaError) as e:
            fn()
        return e.value.code

    assert code_of(lambda: twa.twa_project(ctx, P32, g[1:D + 1], c, ws)) == twa.TWA_ERR_MISALIGNED
    assert code_of(lambda: twa.twa_project(ctx, P32, g[:D], c, ws[:16])) == twa.TWA_ERR_WORKSPACE
    assert code_of(lambda: twa.twa_quantize_basis(ctx, P32, 5, ws)) == twa.TWA_ERR_UNSUPPORTED
    bad = twa.basis_from_tensor(P, D)
    bad.desc.n = 0
    assert code_of(lambda: twa.twa_project(ctx, bad, g[:D], c, ws)) == twa.TWA_ERR_INVALID_ARG
    bad.desc.n = twa.TWA_MAX_N + 1
    assert code_of(lambda: twa.twa_project(ctx, bad, g[:D], c, ws)) == twa.TWA_ERR_UNSUPPORTED
    bad.desc.n = n
    bad.desc.col_stride = 4 * D - 8
    assert code_of(lambda: twa.twa_project(ctx, bad, g[:D], c, ws)) in (
        twa.TWA_ERR_MISALIGNED, twa.TWA_ERR_INVALID_ARG)
    wide = torch.zeros((twa.TWA_MAX_N + 1, 16), device=DEV)
    assert code_of(lambda: twa.twa_build_basis(ctx, wide, 16, torch.zeros(16, device=DEV), ws)) == \
        twa.TWA_ERR_UNSUPPORTED
    # the one-call build: a width it does not have, too many columns, a workspace too small -- all before any launch
    W = random_basis(D, n, 2)
    before = W.clone()
    wbar = torch.zeros(D, device=DEV)
    assert code_of(lambda: twa.twa_build_quantized(ctx, W, D, wbar, [8, 5], ws)) == twa.TWA_ERR_UNSUPPORTED
    assert code_of(lambda: twa.twa_build_quantized(ctx, W, D, wbar, [8], ws[:16])) == twa.TWA_ERR_WORKSPACE
    assert code_of(lambda: twa.twa_build_quantized(ctx, wide, 16, torch.zeros(16, device=DEV), [8], ws)) == \
        twa.TWA_ERR_UNSUPPORTED
    assert torch.equal(W, before)
    status_ok(ctx)


# ------------------------------------------------------------------ row-chunked build
def _chunked_build(ctx, W, D, bits, chunk_rows, want_q32=True):
    n = W.shape[0]
    bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=DEV)
    wbar = torch.full((D + 4,), 9.0, device=DEV)
    q32 = torch.zeros((n, inputs.padded_ld(D, 4)), device=DEV) if want_q32 else None
    Pq = twa.new_quantised_basis(D, n, bits, DEV) if bits != 32 else None
    starts = list(range(0, D, chunk_rows))
    twa.twa_build_begin(ctx, D, n, wbar, bws)
    for p in range(4 if bits != 32 else 3):
        order = starts if p % 2 == 0 else starts[::-1]          # any order within a pass
        for r0 in order:
            rows = min(chunk_rows, D - r0)
            twa.twa_build_feed(ctx, p, W[:, r0:], r0, rows, Pq=Pq if p == 3 else None,
                               q32_out=q32[:, r0:] if p >= 2 else None)
        twa.twa_build_end_pass(ctx, p, bits if p == 2 else 0, Pq if p == 2 else None)
    return wbar, q32, Pq


@pytest.mark.parametrize("D,n,chunk_rows", [(300007, 20, 131072), (70001, 33, 8192), (5000, 3, 1024),
                                           (260000, 64, 65536)])
def test_chunked_build_matches_oracle_and_resident_build(env, D, n, chunk_rows):
    ctx, ws = env
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 31, DEV, ld=inputs.padded_ld(D, 4))
    A = host_cols(W, D).copy()
    wbar, q32, _ = _chunked_build(ctx, W, D, 32, chunk_rows)
    status_ok(ctx)
    np.testing.assert_array_equal(wbar[:D].cpu().numpy(), orc.mean(A).astype(np.float32))
    assert torch.all(wbar[D:] == 9.0)
    Qg = host_cols(q32, D).astype(np.float64)
    assert np.max(np.abs(Qg.T @ Qg - np.eye(n))) <= 1e-5
    Q, _, bad = orc.cgs2(A)
    assert bad is None
    kappa = np.linalg.cond(A.astype(np.float64))
    assert np.max(np.linalg.norm(Qg - Q, axis=0)) <= 1e-6 + 100 * kappa * np.finfo(np.float64).eps
    assert torch.all(q32[:, D:] == 0)
    # the resident float32 Gram-Schmidt build gives the same basis up to its float32 rounding
    W2 = W.clone()
    wbar2 = torch.empty(D, device=DEV)
    twa.twa_build_basis(ctx, W2, D, wbar2, ws)
    status_ok(ctx)
    assert torch.equal(wbar2, wbar[:D])
    assert np.max(np.linalg.norm(host_cols(W2, D) - Qg, axis=0)) <= 10 * kappa * np.finfo(np.float32).eps


@pytest.mark.parametrize("bits", [8, 4])
def test_chunked_build_codes_are_the_quantiser_of_its_float32_rows(env, bits):
    ctx, ws = env
    D, n, chunk_rows = 150001, 12, 32768
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 32, DEV, ld=inputs.padded_ld(D, 4))
    wbar, q32, Pq = _chunked_build(ctx, W, D, bits, chunk_rows)
    status_ok(ctx)
    codes_g, s_g = twa.twa_basis_export(ctx, Pq)
    codes_o, s_o = orc.quantize(np.asfortranarray(host_cols(q32, D)), bits)
    np.testing.assert_array_equal(s_g.cpu().numpy(), s_o)
    np.testing.assert_array_equal(codes_g.cpu().numpy(), orc.pack_codes(codes_o, bits))
    # identical to quantising the float32 rows with the resident quantiser, padding included
    Pq2 = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(q32, D), bits, ws)
    assert torch.equal(Pq.data, Pq2.data) and torch.equal(Pq.scales, Pq2.scales)
    # and usable by the step kernels
    g = inputs.gradient(D, 1e-3, 5, 0, torch.float32, DEV)
    c = torch.empty(n, device=DEV)
    twa.twa_project(ctx, Pq, g, c, ws)
    c_ref = orc.project(codes_o, s_o, g.cpu().numpy())
    assert rel(c.cpu().numpy(), c_ref) <= TOL
    status_ok(ctx)


@pytest.mark.parametrize("D,n,chunk_rows", [(150001, 12, 32768), (100, 3, 1024), (600, 2, 1024), (70001, 33, 8192),
                                            (5121, 64, 2048)])
def test_chunked_build_two_widths_in_one_last_pass(env, D, n, chunk_rows):
    """twa_build_feed_codes with the 8-bit and the 4-bit basis together: the bytes of one
    twa_build_feed per basis, padding included -- also where the last segment of the 4-bit columns
    ends later than that of the 8-bit ones -- and the oracle's quantiser on the float32 rows."""
    ctx, ws = env
    W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 36, DEV, ld=inputs.padded_ld(D, 4))
    bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=DEV)
    wbar = torch.empty(D, device=DEV)
    q32 = torch.zeros((n, inputs.padded_ld(D, 4)), device=DEV)
    sep = {bits: twa.new_quantised_basis(D, n, bits, DEV) for bits in (8, 4)}
    both = {bits: twa.new_quantised_basis(D, n, bits, DEV) for bits in (8, 4)}
    for q in list(sep.values()) + list(both.values()):
        q.data.fill_(0xA5)                                    # whatever was there must be overwritten
    starts = list(range(0, D, chunk_rows))
    twa.twa_build_begin(ctx, D, n, wbar, bws)
    for p in range(3):
        for r0 in starts:
            twa.twa_build_feed(ctx, p, W[:, r0:], r0, min(chunk_rows, D - r0), q32_out=q32[:, r0:] if p == 2 else None)
        if p < 2:
            twa.twa_build_end_pass(ctx, p, 0, None)
    for bits in (8, 4):
        twa.twa_build_end_pass(ctx, 2, bits, sep[bits])
        twa.twa_build_end_pass(ctx, 2, bits, both[bits])
    for r0 in starts:
        rows = min(chunk_rows, D - r0)
        for bits in (8, 4):
            twa.twa_build_feed(ctx, 3, W[:, r0:], r0, rows, Pq=sep[bits])
        twa.twa_build_feed_codes(ctx, W[:, r0:], r0, rows, [both[8], both[4]])
    twa.twa_build_end_pass(ctx, 3, 0, None)
    status_ok(ctx)
    for bits in (8, 4):
        assert torch.equal(sep[bits].data, both[bits].data) and torch.equal(sep[bits].scales, both[bits].scales)
        codes_g, s_g = twa.twa_basis_export(ctx, both[bits])
        codes_o, s_o = orc.quantize(np.asfortranarray(host_cols(q32, D)), bits)
        np.testing.assert_array_equal(s_g.cpu().numpy(), s_o)
        np.testing.assert_array_equal(codes_g.cpu().numpy(), orc.pack_codes(codes_o, bits))


def test_chunked_build_reports_rank_deficiency(env):
    ctx, ws = env
    D, n = 20000, 5
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 33, DEV, ld=inputs.padded_ld(D, 4))
    W[3] = W[1] * 0.5
    _chunked_build(ctx, W, D, 32, 4096)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_RANK_DEFICIENT, 3)
    twa.twa_clear_status(ctx)


@pytest.mark.parametrize("segments", [1, 2, 4])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("D,n", [(4099, 33), (70001, 100), (131072, 8)])
def test_tile_segments_knob(env, D, n, bits, segments):
    """Both tile heights of the tensor-pipe kernels, whatever the built-in choice for this n."""
    ctx, ws = env
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_TILE_SEGMENTS, segments)
    try:
        P = random_basis(D, n, 900 + D + n)
        B = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), bits, ws)
        codes, s = twa.twa_basis_export(ctx, B)
        co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
        gen = torch.Generator(device=DEV)
        gen.manual_seed(D + n + bits)
        g = (torch.randn(D, generator=gen, device=DEV) * 1e-4).bfloat16()
        alpha = torch.randn(n, generator=gen, device=DEV)
        base = torch.randn(D, generator=gen, device=DEV)
        c = torch.empty(n, device=DEV)
        w = torch.full((D + 8,), 5.0, device=DEV)
        twa.twa_project(ctx, B, g, c, ws)
        twa.twa_lift(ctx, B, alpha, base, w, ws)
        status_ok(ctx)
        assert rel(c.cpu().numpy(), orc.project(co, so, g.float().cpu().numpy())) <= TOL
        w_ref = orc.lift(co, so, alpha.cpu().numpy(), base.cpu().numpy())
        assert rel(w[:D].cpu().numpy(), w_ref) <= TOL
        assert rel(w[:D].cpu().numpy().astype(np.float64) - base.cpu().numpy(),
                   w_ref - base.cpu().numpy()) <= 1e-4          # P alpha carried by a float32 w
        assert torch.all(w[D:] == 5.0)
    finally:
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_TILE_SEGMENTS, 0)


@pytest.mark.parametrize("segments", [0, 1, 2, 4])
@pytest.mark.parametrize("gdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("D,n", [(2, 1), (4099, 33), (70002, 20), (70001, 20), (131072, 8), (40000, 64), (9000, 128)])
def test_float32_projection_tile_heights(env, D, n, gdt, segments):
    """The float32 projection in tiles of one, two and four 512-byte segments (four: even D only,
    else the library falls back to two), with poison in the padding behind row D - 1 of every column."""
    ctx, ws = env
    P = random_basis(D, n, 4100 + D + n)
    P[:, D:] = float("nan")
    gen = torch.Generator(device=DEV)
    gen.manual_seed(D * 3 + n)
    g = (torch.randn(D, generator=gen, device=DEV) * 1e-3).to(gdt)
    c = torch.full((n + 1,), 7.0, device=DEV)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_TILE_SEGMENTS, segments)
    try:
        twa.twa_project(ctx, twa.basis_from_tensor(P, D), g, c, ws)
    finally:
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_TILE_SEGMENTS, 0)
    status_ok(ctx)
    assert rel(c[:n].cpu().numpy(), orc.project_f32(host_cols(P, D), g.float().cpu().numpy())) <= TOL
    assert c[n].item() == 7.0


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("D,n", [(1, 1), (4099, 33), (70001, 100), (131075, 8), (600001, 32)])
def test_lift_vectors_knob(env, D, n, bits):
    """The lift's ways of moving `base` and the output (loaded and stored by the lanes, or through
    the shared-memory ring and bulk stores) do the same arithmetic: identical bits, all matching the oracle."""
    ctx, ws = env
    P = random_basis(D, n, 1700 + D + n)
    B = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), bits, ws)
    codes, s = twa.twa_basis_export(ctx, B)
    co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
    gen = torch.Generator(device=DEV)
    gen.manual_seed(D + 3 * n + bits)
    alpha = torch.randn(n, generator=gen, device=DEV)
    base = torch.randn(D + 8, generator=gen, device=DEV)
    base[D:] = float("nan")                         # must never reach the output
    out = []
    try:
        for mode in (1, 2, 3):
            twa.twa_set_tuning(ctx, twa.TWA_TUNE_LIFT_VECTORS, mode)
            w = torch.full((D + 8,), 5.0, device=DEV)
            twa.twa_lift(ctx, B, alpha, base[:D], w, ws)
            status_ok(ctx)
            assert torch.all(w[D:] == 5.0)
            out.append(w[:D].clone())
    finally:
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_LIFT_VECTORS, 0)
    assert torch.equal(out[0], out[1]) and torch.equal(out[0], out[2])
    w_ref = orc.lift(co, so, alpha.cpu().numpy(), base[:D].cpu().numpy())
    assert rel(out[0].cpu().numpy(), w_ref) <= TOL


def test_bounded_wait_runs_out_cleanly_and_the_context_stays_usable(env):
    """A wait that nothing satisfies ends after its limit with a status, not a hang or a fault."""
    ctx, ws = env
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_WAIT_LIMIT_MS, 20)
    try:
        twa.twa_selftest_wait(ctx)
        code, detail = twa.twa_get_status(ctx)
        assert code == twa.TWA_ERR_TIMEOUT
    finally:
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_WAIT_LIMIT_MS, 0)
        twa.twa_clear_status(ctx)
    status_ok(ctx)
    D, n = 4099, 5
    P = random_basis(D, n, 4)
    B = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), 8, ws)
    g = torch.randn(D, device=DEV)
    c = torch.empty(n, device=DEV)
    twa.twa_project(ctx, B, g, c, ws)
    codes, s = twa.twa_basis_export(ctx, B)
    co = orc.unpack_codes(codes.cpu().numpy(), D, 8)
    assert rel(c.cpu().numpy(), orc.project(co, s.cpu().numpy(), g.cpu().numpy())) <= TOL
    status_ok(ctx)


# ------------------------------------------------------------------ panel build against the column-wise build
@pytest.mark.parametrize("D,n,step", [(50001, 24, 0.005), (50001, 24, 0.0002), (120007, 77, 0.002), (9001, 9, 0.01)])
def test_panel_build_agrees_with_column_build_and_oracle(env, D, n, step):
    ctx, ws = env
    wbar = torch.empty(D, device=DEV)
    out = {}
    for mode in (1, 2, 0):       # 1: column by column; 2: panels of 8, sweeps inside; 0: panels, Gram form inside (default)
        W = inputs.trajectory_candidates(D, n, step, 0.001, 31, DEV, ld=inputs.padded_ld(D, 4))
        A = host_cols(W, D).copy()
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, mode)
        try:
            twa.twa_build_basis(ctx, W, D, wbar, ws)
        finally:
            twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, 0)
        status_ok(ctx)
        out[mode] = host_cols(W, D).astype(np.float64)
    Q, _, bad = orc.cgs2(A)
    assert bad is None
    kappa = np.linalg.cond(A.astype(np.float64))
    for mode, Pg in out.items():
        assert np.max(np.abs(Pg.T @ Pg - np.eye(n))) <= 1e-5, mode
        assert np.max(np.linalg.norm(Pg - Q, axis=0)) <= 10 * kappa * np.finfo(np.float32).eps, mode
        T = Pg.T @ A.astype(np.float64)
        assert np.all(np.diag(T) > 0) and np.max(np.abs(np.tril(T, -1))) <= 2e-5 * np.max(np.abs(T))
    # the schedules reach the same vectors to the accuracy each reaches the oracle
    for mode in (0, 2):
        assert np.max(np.linalg.norm(out[mode] - out[1], axis=0)) <= 20 * kappa * np.finfo(np.float32).eps, mode


def test_build_quantized_with_a_dependent_candidate(env):
    """A candidate that repeats an earlier one: both forms of the call report it, zero its column and
    give it the scale 0 and the codes 0."""
    ctx, ws = env
    D, n = 30011, 21
    ld = inputs.padded_ld(D, 4)
    outs = []
    for one_call in (False, True):
        W = inputs.trajectory_candidates(D, n, 0.005, 0.001, 78, DEV, ld=ld)
        W[13] = W[4]
        wbar = torch.empty(D, device=DEV)
        if one_call:
            P32, (q8, q4) = twa.twa_build_quantized(ctx, W, D, wbar, [8, 4], ws)
        else:
            P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
            q8, q4 = twa.twa_quantize_basis(ctx, P32, 8, ws), twa.twa_quantize_basis(ctx, P32, 4, ws)
        code, detail = twa.twa_get_status(ctx)
        assert (code, detail) == (twa.TWA_ERR_RANK_DEFICIENT, 13)
        twa.twa_clear_status(ctx)
        assert torch.all(W[13] == 0)
        for q in (q8, q4):
            codes, scales = twa.twa_basis_export(ctx, q)
            assert scales[13].item() == 0.0 and torch.all(codes[13] == 0)
        outs.append((W, q8.data, q8.scales, q4.data, q4.scales))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("D,n", [(1, 1), (5003, 3), (70001, 33), (300007, 20), (40001, 128)])
def test_build_quantized_equals_build_then_quantize_bit_for_bit(env, D, n, mode):
    """One call for mean, basis and both storage widths: the column maxima it takes while the build
    writes its last pass are those a pass over the finished basis finds, so basis, scales and codes
    are those of twa_build_basis followed by twa_quantize_basis -- and the codes are the oracle's
    quantiser applied to that basis."""
    ctx, ws = env
    ld = inputs.padded_ld(D, 4)
    wbar_a, wbar_b = torch.empty(D, device=DEV), torch.empty(D, device=DEV)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, mode)
    try:
        Wa = inputs.trajectory_candidates(D, n, 0.005, 0.001, 77, DEV, ld=ld)
        P32a = twa.twa_build_basis(ctx, Wa, D, wbar_a, ws)
        qa = [twa.twa_quantize_basis(ctx, P32a, bits, ws) for bits in (8, 4)]
        Wb = inputs.trajectory_candidates(D, n, 0.005, 0.001, 77, DEV, ld=ld)
        P32b, qb = twa.twa_build_quantized(ctx, Wb, D, wbar_b, [8, 4], ws)
    finally:
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, 0)
    status_ok(ctx)
    assert torch.equal(Wa, Wb) and torch.equal(wbar_a, wbar_b)
    assert (P32b.D, P32b.n, P32b.bits, P32b.col_stride) == (D, n, 32, 4 * ld)
    P_h = host_cols(Wb, D)
    for bits, A, B in zip((8, 4), qa, qb):
        assert (B.D, B.n, B.bits, B.col_stride) == (D, n, bits, twa.twa_basis_col_stride(D, bits))
        ca, sa = twa.twa_basis_export(ctx, A)
        cb, sb = twa.twa_basis_export(ctx, B)
        assert torch.equal(sa, sb) and torch.equal(ca, cb)
        assert torch.equal(A.data, B.data)                    # padding included
        codes_o, scales_o = orc.quantize(np.asfortranarray(P_h), bits)
        np.testing.assert_array_equal(sb.cpu().numpy(), scales_o)
        np.testing.assert_array_equal(cb.cpu().numpy(), orc.pack_codes(codes_o, bits))


@pytest.fixture(params=[0, 2], ids=["gram-in-panel", "sweeps-in-panel"])
def panel_mode(request, env):
    ctx, _ = env
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, request.param)
    yield request.param
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, 0)


def test_panel_build_finds_dependence_across_and_inside_panels(env, panel_mode):
    ctx, ws = env
    D, n = 30001, 20
    wbar = torch.empty(D, device=DEV)
    for bad_col, src in ((13, 3), (14, 9), (7, 0), (0, None), (19, 18)):   # earlier panel; same panel; first panel; zero first column; last
        W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 2, DEV, ld=inputs.padded_ld(D, 4))
        W[bad_col] = W[src] * -2.0 if src is not None else 0.0
        twa.twa_build_basis(ctx, W, D, wbar, ws)
        code, detail = twa.twa_get_status(ctx)
        assert (code, detail) == (twa.TWA_ERR_RANK_DEFICIENT, bad_col)
        twa.twa_clear_status(ctx)
        Pg = host_cols(W, D).astype(np.float64)
        keep = [j for j in range(n) if j != bad_col]
        assert np.all(Pg[:, bad_col] == 0)                 # the dependent column is zeroed, the rest is a basis
        assert np.max(np.abs(Pg[:, keep].T @ Pg[:, keep] - np.eye(n - 1))) <= 1e-5
    W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 2, DEV, ld=inputs.padded_ld(D, 4))
    W[11, 222] = float("nan")
    twa.twa_build_basis(ctx, W, D, wbar, ws)
    code, detail = twa.twa_get_status(ctx)
    assert code == twa.TWA_ERR_NONFINITE and 8 <= detail <= 15      # reported for the panel that holds it
    twa.twa_clear_status(ctx)


@pytest.mark.parametrize("ratio,deficient", [(3e-5, False), (3e-6, True)])
def test_nearly_dependent_column_inside_a_panel_all_schedules_agree(env, ratio, deficient):
    """One candidate of the second panel is its neighbour plus a small step, so that its remainder
    after orthogonalisation is `ratio` times its length: just above the float32 rank rule (1e-5)
    the three schedules and the oracle give the same orthonormal basis, just below it all three
    report that column (the oracle, run with the same rule, names the same one)."""
    ctx, ws = env
    D, n, col = 60001, 20, 11
    wbar = torch.empty(D, device=DEV)

    def candidates():
        W = inputs.trajectory_candidates(D, n, 0.01, 0.002, 5, DEV, ld=inputs.padded_ld(D, 4))
        gen = torch.Generator(device=DEV)
        gen.manual_seed(77)
        xi = torch.randn(D, generator=gen, device=DEV)
        W[col, :D] = W[col - 1, :D] + xi * (ratio * W[col - 1, :D].norm() / xi.norm())
        return W

    A = host_cols(candidates(), D).copy()
    Q, _, bad = orc.cgs2(A, rel_tol=1e-5)                       # the GPU build's rule
    assert (bad == col) if deficient else (bad is None)
    kappa = np.linalg.cond(A.astype(np.float64))
    out = {}
    for mode in (1, 2, 0):
        W = candidates()
        twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, mode)
        try:
            twa.twa_build_basis(ctx, W, D, wbar, ws)
        finally:
            twa.twa_set_tuning(ctx, twa.TWA_TUNE_BUILD_PANEL, 0)
        code, detail = twa.twa_get_status(ctx)
        twa.twa_clear_status(ctx)
        Pg = host_cols(W, D).astype(np.float64)
        if deficient:
            assert (code, detail) == (twa.TWA_ERR_RANK_DEFICIENT, col), mode
            keep = [j for j in range(n) if j != col]
            assert np.all(Pg[:, col] == 0)
            assert np.max(np.abs(Pg[:, keep].T @ Pg[:, keep] - np.eye(n - 1))) <= 1e-5, mode
        else:
            assert code == 0, (mode, code, detail)
            assert np.max(np.abs(Pg.T @ Pg - np.eye(n))) <= 1e-5, mode
            assert np.max(np.linalg.norm(Pg - Q, axis=0)) <= 10 * kappa * np.finfo(np.float32).eps, mode
        out[mode] = Pg
    if not deficient:
        for mode in (0, 2):
            assert np.max(np.linalg.norm(out[mode] - out[1], axis=0)) <= 20 * kappa * np.finfo(np.float32).eps


def test_step_keeps_the_coefficients_when_the_gradient_is_not_finite(env):
    """alpha is state that outlives a call: a step whose projection is not finite reports
    TWA_ERR_NONFINITE, leaves alpha as it was and lifts w from that alpha; after clearing the status
    the next step continues as if the bad one had not been made."""
    ctx, ws = env
    D, n = 20011, 12
    for bits in (8, 32):
        P = random_basis(D, n, 21)
        B = twa.basis_from_tensor(P, D)
        if bits != 32:
            B = twa.twa_quantize_basis(ctx, B, bits, ws)
        wbar = torch.randn(D, device=DEV)
        alpha = torch.zeros(n, device=DEV)
        w = torch.empty(D, device=DEV)
        g = inputs.gradient(D, 1e-3, 4, 0, torch.float32, DEV)
        twa.twa_step(ctx, B, g, 0.1, 0.0, alpha, wbar, w, ws)
        status_ok(ctx)
        before, w_before = alpha.clone(), w.clone()
        g_bad = g.clone()
        g_bad[1234] = float("nan")
        c = torch.empty(n, device=DEV)
        twa.twa_step(ctx, B, g_bad, 0.1, 0.0, alpha, wbar, w, ws, c_out=c)
        code, _ = twa.twa_get_status(ctx)
        assert code == twa.TWA_ERR_NONFINITE
        assert torch.isnan(c).any()
        assert torch.equal(alpha, before)
        if bits != 32:
            assert torch.equal(w, w_before)                 # lifted from the unchanged alpha
        twa.twa_clear_status(ctx)
        # the same good step twice from the same state gives the same alpha as stepping once more
        ref = before.clone()
        twa.twa_step(ctx, B, g, 0.1, 0.0, ref, wbar, torch.empty(D, device=DEV), ws)
        twa.twa_step(ctx, B, g, 0.1, 0.0, alpha, wbar, w, ws)
        status_ok(ctx)
        assert torch.equal(alpha, ref)


# ------------------------------------------------------------------ the digit cut of the gradient at its limits
def _digit_cut_bound(co, so, g64, rows_per_block, three_bytes):
    """Bound of the projection's error from cutting g into byte digits: every value of a warp's block
    of rows carries an absolute error of at most 2^-23 (three bytes) or 2^-31 (four) of the power of two
    above the block's largest magnitude, so |delta c_j| <= sum over blocks of that times sum |p~[r, j]|."""
    D, n = co.shape
    bound = np.zeros(n)
    eps = 2.0 ** -23 if three_bytes else 2.0 ** -31
    absP = np.abs(co.astype(np.float64)) * np.abs(so.astype(np.float64))[None, :]
    for r0 in range(0, D, rows_per_block):
        m = np.max(np.abs(g64[r0:r0 + rows_per_block]))
        if m > 0:
            bound += eps * 2.0 ** np.ceil(np.log2(m) + 1e-12) * absP[r0:r0 + rows_per_block].sum(axis=0)
    return bound


@pytest.mark.parametrize("kind", ["heavy_tail", "one_outlier_per_block", "tiny", "huge", "ties"])
@pytest.mark.parametrize("gdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bits", [8, 4])
def test_projection_digit_cut_on_hard_gradients(env, bits, gdt, kind):
    """Gradients that stress the block-fixed-point cut: heavy tails (Student t, 1.5 degrees of freedom),
    one value 2^20 times the rest in every block of rows, magnitudes near the ends of the float range, and
    values that sit exactly on rounding ties of the cut.  The result stays within the stated relative bound
    where the coefficients are well conditioned, and always within the bound derived from the cut plus the
    float32 accumulation term."""
    ctx, ws = env
    D, n = 70001, 33
    P = random_basis(D, n, 303)
    B = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(P, D), bits, ws)
    codes, s = twa.twa_basis_export(ctx, B)
    co, so = orc.unpack_codes(codes.cpu().numpy(), D, bits), s.cpu().numpy()
    rng = np.random.default_rng(17)
    if kind == "heavy_tail":
        g = rng.standard_t(1.5, size=D) * 1e-3
    elif kind == "one_outlier_per_block":
        g = rng.standard_normal(D) * 1e-3
        g[::64] *= 2.0 ** 20
    elif kind == "tiny":
        g = rng.standard_normal(D) * 1e-30
    elif kind == "huge":
        g = rng.standard_normal(D) * 1e30
    else:
        # multiples of 2^-12 with a block maximum of 1023.5: the cut scales them by 2^12 (bfloat16: exact
        # integers) -- every value is an exact integer or half-integer of the digit grid
        g = rng.integers(-2048, 2049, size=D) * 2.0 ** -2
        g[::128] = 1023.5
    gt = torch.from_numpy(g.astype(np.float32)).to(DEV).to(gdt)
    g64 = gt.float().cpu().numpy().astype(np.float64)
    c = torch.empty(n, device=DEV)
    twa.twa_project(ctx, B, gt, c, ws)
    status_ok(ctx)
    c_ref = orc.project(co, so, g64)
    err = np.abs(c.cpu().numpy().astype(np.float64) - c_ref)
    # a warp cuts 32 * KT bytes of a column with one scale: at n = 33 (KT = 2) 64 rows at 8 bits, 128 at 4
    cut = _digit_cut_bound(co, so, g64, 64 * 8 // bits, gdt == torch.bfloat16)
    accumulate = 4e-6 * (np.abs(co.astype(np.float64)) * np.abs(so.astype(np.float64))[None, :]).T @ np.abs(g64)
    assert np.all(err <= cut + accumulate + 1e-45)
    assert rel(c.cpu().numpy(), c_ref) <= TOL
