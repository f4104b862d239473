"""Full-size parity on the five synthetic workloads, through the same calls and launch
configuration the benchmark times.

The two small workloads are compared with the oracle element by element.  For the large
ones the oracle checks what it can compute in seconds on the same bytes: sampled columns of
the codes and of the projection, sampled row ranges of the lift, and the invariants of the
basis on sampled columns (unit norm, mutual orthogonality, triangular relation with the
candidates).  Bounds as everywhere: codes and scales bit-exact, 1e-5 relative L2 for
projection and lift, 1e-5 for orthonormality.
"""

import numpy as np
import pytest
import torch

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import inputs, twa

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
TOL = 1e-5
LR = 0.1


@pytest.fixture(scope="module")
def env():
    torch.cuda.set_device(0)
    ctx = twa.twa_create(0)
    ws = twa.new_workspace(DEV)
    yield ctx, ws
    torch.cuda.synchronize()
    twa.twa_destroy(ctx)
    torch.cuda.empty_cache()


def rel(x, y):
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    return np.linalg.norm(x - y) / np.linalg.norm(y)


def status_ok(ctx):
    code, detail = twa.twa_get_status(ctx)
    assert code == 0, (twa.twa_strerror(code), detail)


def host_col(t, j, D):
    return t[j, :D].cpu().numpy()


def oracle_project_chunked(codes, scales, g, chunk=1 << 24):
    """oracle.project summed over row chunks (it is linear in the rows)."""
    D = codes.shape[0]
    c = np.zeros(codes.shape[1])
    for r0 in range(0, D, chunk):
        c += orc.project(codes[r0:r0 + chunk], scales, g[r0:r0 + chunk])
    return c


def check_step_sampled(ctx, ws, wl, Pq, wbar, bits, col_blocks, row_ranges):
    """One fused step from alpha = 0 on the full workload; oracle on sampled columns / rows."""
    D, n = wl.D, wl.n
    g = wl.gradient(0, DEV)
    alpha = torch.zeros(n, device=DEV)
    w = torch.empty(D, device=DEV)
    c = torch.empty(n, device=DEV)
    twa.twa_step(ctx, Pq, g, LR, 0.0, alpha, wbar, w, ws, c_out=c)
    status_ok(ctx)
    g_host = g.float().cpu().numpy()
    c_host, a_host = c.cpu().numpy(), alpha.cpu().numpy()
    seg = 512 * 8 // bits
    for j0 in col_blocks:
        cols = min(8, n - j0)
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(Pq, col0=j0, cols=cols))
        co = orc.unpack_codes(codes.cpu().numpy(), D, bits)
        so = s.cpu().numpy()
        pick = [0, cols - 1] if cols > 1 else [0]
        c_ref = oracle_project_chunked(co[:, pick], so[pick], g_host)
        assert rel(c_host[[j0 + k for k in pick]], c_ref) <= TOL
        np.testing.assert_allclose(a_host[[j0 + k for k in pick]], -LR * c_ref, rtol=2e-5, atol=0)
        del codes, co
    for r0, rows in row_ranges:
        assert r0 % seg == 0
        rows = min(rows, D - r0)
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=r0, rows=rows))
        co = orc.unpack_codes(codes.cpu().numpy(), rows, bits)
        base = wbar[r0:r0 + rows].cpu().numpy()
        w_ref = orc.lift(co, s.cpu().numpy(), a_host.astype(np.float64), base)
        w_got = w[r0:r0 + rows].cpu().numpy()
        assert rel(w_got, w_ref) <= TOL
        assert np.max(np.abs(w_got - w_ref.astype(np.float32))) <= 4 * np.spacing(np.float32(np.abs(w_ref).max()))
    # the lift alone, without the base point: the bound that is not carried by w_bar
    twa.twa_lift(ctx, Pq, alpha, None, w, ws)
    for r0, rows in row_ranges[:1]:
        rows = min(rows, D - r0)
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=r0, rows=rows))
        co = orc.unpack_codes(codes.cpu().numpy(), rows, bits)
        assert rel(w[r0:r0 + rows].cpu().numpy(), orc.lift(co, s.cpu().numpy(), a_host.astype(np.float64), None)) <= TOL
    status_ok(ctx)


def check_codes_sampled(ctx, P32, Pq, bits, cols):
    """Codes and scales of sampled columns, bit-exact against the oracle's quantiser applied to
    the GPU's own float32 basis column."""
    D = P32.D
    for j in cols:
        j0 = j - j % 8
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(Pq, col0=j0, cols=min(8, Pq.n - j0)))
        col = P32.data[j, :D].cpu().numpy().reshape(-1, 1)
        co, so = orc.quantize(np.asfortranarray(col), bits)
        assert s[j - j0].item() == so[0]
        np.testing.assert_array_equal(codes[j - j0].cpu().numpy(), orc.pack_codes(co, bits)[0])


def check_basis_sampled(W_basis, A_regen, D, cols):
    """Unit norm and mutual orthogonality of sampled basis columns, and zero projection of an
    earlier candidate on a later basis vector (A = Q R with R upper triangular)."""
    Q = [host_col(W_basis, j, D).astype(np.float64) for j in cols]
    for a in range(len(cols)):
        assert abs(np.dot(Q[a], Q[a]) - 1.0) <= TOL
        for b in range(a):
            assert abs(np.dot(Q[a], Q[b])) <= TOL
    for a in range(1, len(cols)):
        early = host_col(A_regen, cols[a - 1], D).astype(np.float64)
        assert abs(np.dot(Q[a], early)) <= 2e-5 * np.linalg.norm(early)      # q_j is orthogonal to w_i, i < j
        late = host_col(A_regen, cols[a], D).astype(np.float64)
        assert np.dot(Q[a], late) > 0                                        # positive diagonal of R


# ------------------------------------------------------------------ tiny: element by element
def test_workload_tiny_float32_basis(env):
    ctx, ws = env
    wl = inputs.WORKLOADS["tiny"]
    D, n = wl.D, wl.n
    W = wl.candidates(DEV)
    A = W[:, :D].cpu().numpy().T.copy()
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    status_ok(ctx)
    Pg = W[:, :D].cpu().numpy().T
    Q, _, bad = orc.cgs2(A)
    assert bad is None
    Pg64 = Pg.astype(np.float64)
    assert np.max(np.abs(Pg64.T @ Pg64 - np.eye(n))) <= TOL
    kappa = np.linalg.cond(A.astype(np.float64))
    assert np.max(np.linalg.norm(Pg64 - Q, axis=0)) <= 10 * kappa * np.finfo(np.float32).eps
    np.testing.assert_array_equal(wbar.cpu().numpy(), orc.mean(A).astype(np.float32))
    g = wl.gradient(0, DEV)
    alpha = torch.zeros(n, device=DEV)
    w = torch.empty(D, device=DEV)
    c = torch.empty(n, device=DEV)
    twa.twa_step(ctx, P32, g, LR, 0.0, alpha, wbar, w, ws, c_out=c)      # alpha from one SGD step
    status_ok(ctx)
    a_o, w_o, c_o = orc.step_f32(Pg, g.cpu().numpy(), np.zeros(n), wbar.cpu().numpy(), LR)
    assert rel(c.cpu().numpy(), c_o) <= TOL
    assert rel(alpha.cpu().numpy(), a_o) <= TOL
    assert rel(w.cpu().numpy(), w_o) <= TOL
    twa.twa_lift(ctx, P32, alpha, None, w, ws)
    assert rel(w.cpu().numpy(), orc.lift_f32(Pg, alpha.cpu().numpy().astype(np.float64), None)) <= TOL


# ------------------------------------------------------------------ ResNet-18-sized: element by element
def test_workload_resnet18_float32_and_int8(env):
    ctx, ws = env
    wl = inputs.WORKLOADS["resnet18"]
    D, n = wl.D, wl.n
    W = wl.candidates(DEV)
    A = W[:, :D].cpu().numpy().T.copy()
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    status_ok(ctx)
    Pg = W[:, :D].cpu().numpy().T
    np.testing.assert_array_equal(wbar.cpu().numpy(), orc.mean(A).astype(np.float32))
    G = np.zeros((n, n))
    for r0 in range(0, D, 1 << 21):                      # float64 Gram, chunk-streamed
        blk = Pg[r0:r0 + (1 << 21)].astype(np.float64)
        G += blk.T @ blk
    assert np.max(np.abs(G - np.eye(n))) <= TOL
    Q, _, bad = orc.cgs2(A)
    assert bad is None
    GA = np.zeros((n, n))
    for r0 in range(0, D, 1 << 21):
        blk = A[r0:r0 + (1 << 21)].astype(np.float64)
        GA += blk.T @ blk
    ev = np.linalg.eigvalsh(GA)
    kappa = float(np.sqrt(ev[-1] / ev[0]))               # condition number of the candidates
    assert max(np.linalg.norm(Pg[:, j].astype(np.float64) - Q[:, j]) for j in range(n)) <= \
        10 * kappa * np.finfo(np.float32).eps
    del Q, A
    Pq = twa.twa_quantize_basis(ctx, P32, 8, ws)
    codes_g, s_g = twa.twa_basis_export(ctx, Pq)
    codes_o, s_o = orc.quantize(np.asfortranarray(Pg), 8)
    np.testing.assert_array_equal(s_g.cpu().numpy(), s_o)
    np.testing.assert_array_equal(codes_g.cpu().numpy(), orc.pack_codes(codes_o, 8))
    for basis, ostep in ((P32, lambda g, a: orc.step_f32(Pg, g, a, wbar.cpu().numpy(), LR)),
                         (Pq, lambda g, a: orc.step(codes_o, s_o, g, a, wbar.cpu().numpy(), LR))):
        alpha = torch.zeros(n, device=DEV)
        w = torch.empty(D, device=DEV)
        c = torch.empty(n, device=DEV)
        a_o = np.zeros(n)
        for t in range(3):                                # fresh gradient every step
            g = wl.gradient(t, DEV)
            twa.twa_step(ctx, basis, g, LR, 0.0, alpha, wbar, w, ws, c_out=c)
            a_o, w_o, c_o = ostep(g.cpu().numpy(), a_o)
            assert rel(c.cpu().numpy(), c_o) <= TOL
            assert rel(alpha.cpu().numpy(), a_o) <= TOL
            assert rel(w.cpu().numpy(), w_o) <= TOL
        status_ok(ctx)


# ------------------------------------------------------------------ ResNet-50- and ViT-B-sized: sampled
@pytest.mark.parametrize("name,bits_list", [("resnet50", (8,)), ("vitb16", (8, 4))])
def test_workload_resident_build_sampled(env, name, bits_list):
    ctx, ws = env
    wl = inputs.WORKLOADS[name]
    D, n = wl.D, wl.n
    W = wl.candidates(DEV)
    wbar = torch.empty(D, device=DEV)
    P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    status_ok(ctx)
    A = wl.candidates(DEV)                               # the same candidates again (the build is in place)
    cols = [0, 1, n // 2, n - 2, n - 1]
    check_basis_sampled(W, A, D, cols)
    # w_bar on sampled rows against the oracle's mean
    for r0 in (0, D // 2, D - 4099):
        blk = A[:, r0:r0 + 4099].cpu().numpy().T
        np.testing.assert_array_equal(wbar[r0:r0 + 4099].cpu().numpy(), orc.mean(blk).astype(np.float32))
    del A
    torch.cuda.empty_cache()
    for bits in bits_list:
        seg = 512 * 8 // bits
        Pq = twa.twa_quantize_basis(ctx, P32, bits, ws)
        status_ok(ctx)
        check_codes_sampled(ctx, P32, Pq, bits, [0, n // 2 + 1, n - 1])
        last = (D // seg) * seg                           # the ragged last segment
        check_step_sampled(ctx, ws, wl, Pq, wbar, bits, col_blocks=[0, ((n - 1) // 8) * 8],
                           row_ranges=[(0, 2 * seg), ((D // 2 // seg) * seg, 3 * seg), (last, seg)])
        del Pq
        torch.cuda.empty_cache()


# ------------------------------------------------------------------ 1.3 B-sized: chunked build, sampled
def test_workload_decoder_chunked_build_sampled(env):
    ctx, ws = env
    wl = inputs.WORKLOADS["decoder1p3b"]
    D, n, bits = wl.D, wl.n, 8
    CH = inputs.CHUNK_ROWS
    starts = list(range(0, D, CH))
    sampled = {starts[0]: None, starts[len(starts) // 2]: None, starts[-1]: None}
    bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=DEV)
    wbar = torch.empty(D, device=DEV)
    Pq = twa.new_quantised_basis(D, n, bits, DEV)
    buf = torch.empty((n, CH), device=DEV)
    qbuf = torch.empty((n, CH), device=DEV)
    twa.twa_build_begin(ctx, D, n, wbar, bws)
    for p in range(4):
        for r0 in starts:
            rows = min(CH, D - r0)
            inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, DEV, row0=r0, rows=rows, out=buf[:, :rows])
            keep = p == 3 and r0 in sampled
            twa.twa_build_feed(ctx, p, buf, r0, rows, Pq=Pq if p == 3 else None, q32_out=qbuf if keep else None)
            if keep:
                sampled[r0] = (qbuf[:, :rows].cpu().numpy().T.copy(), buf[:, :rows].cpu().numpy().T.copy())
        twa.twa_build_end_pass(ctx, p, bits if p == 2 else 0, Pq if p == 2 else None)
    status_ok(ctx)
    del buf, qbuf, bws
    torch.cuda.empty_cache()
    scales = Pq.scales.cpu().numpy()
    for r0, (q32, a_rows) in sampled.items():
        rows = q32.shape[0]
        # codes of the chunk = the oracle's encoder on the chunk's float32 rows with the global scales
        codes, _ = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=r0, rows=rows))
        co = orc.encode(np.asfortranarray(q32), scales, bits)
        np.testing.assert_array_equal(codes.cpu().numpy(), orc.pack_codes(co, bits))
        assert np.all(np.abs(q32).max(axis=0) <= scales * 127 * (1 + 1e-6))
        # w_bar rows = the oracle's mean of the candidate rows
        np.testing.assert_array_equal(wbar[r0:r0 + rows].cpu().numpy(), orc.mean(a_rows).astype(np.float32))
        # rows of Q are rows of A times one upper-triangular matrix: the same M for every chunk
        if r0 == 0:
            M0, *_ = np.linalg.lstsq(a_rows[:65536].astype(np.float64), q32[:65536].astype(np.float64), rcond=None)
            assert np.max(np.abs(np.tril(M0, -1))) <= 1e-3 * np.max(np.abs(M0))
            assert np.all(np.diag(M0) > 0)
        else:
            resid = a_rows[:65536].astype(np.float64) @ M0 - q32[:65536]
            assert np.linalg.norm(resid) <= 1e-5 * np.linalg.norm(q32[:65536])
    sampled.clear()
    # unit columns: the dequantised basis has norm 1 up to the quantisation error (oracle on one column)
    codes, s = twa.twa_basis_export(ctx, twa.basis_view(Pq, col0=24, cols=8))
    col = codes[7].cpu().numpy().view(np.int8)[:D].astype(np.float64)
    assert abs(np.sqrt(np.dot(col, col)) * float(s[7]) - 1.0) <= 2e-3
    del codes
    torch.cuda.empty_cache()
    seg = 512
    check_step_sampled(ctx, ws, wl, Pq, wbar, bits, col_blocks=[24],
                       row_ranges=[(0, 2 * seg), ((D // 2 // seg) * seg, 2 * seg), (D - seg, seg)])


# ------------------------------------------------------------------ the layer-wise construction, full size
def _unpack_rows(packed, r0, r1, bits):
    """Unsigned codes of flat rows r0..r1-1 (r0 even) from the canonical export, shape (rows, n)."""
    if bits == 8:
        return np.asfortranarray(packed[:, r0:r1].cpu().numpy().T)
    b = packed[:, r0 // 2:(r1 + 1) // 2].cpu().numpy()
    inter = np.empty((b.shape[0], 2 * b.shape[1]), dtype=np.uint8)
    inter[:, 0::2], inter[:, 1::2] = b & 0xF, b >> 4
    return np.asfortranarray(inter[:, :r1 - r0].T)


@pytest.mark.parametrize("name,bits_list", [("resnet50", (8,)), ("vitb16", (8, 4))])
def test_workload_layerwise_sampled(env, name, bits_list):
    """The paper's default construction on the workload's own layer partition: per-layer factors
    and sampled codes bit-exact, one layer-wise step checked on sampled layers, columns and rows."""
    ctx, _ = env
    wl = inputs.WORKLOADS[name]
    D, n = wl.D, wl.n
    layers = inputs.layer_offsets(name)
    L = len(layers) - 1
    sizes = np.diff(layers)
    W = wl.candidates(DEV)
    wbar = torch.empty(D, device=DEV)
    lws = twa.new_layered_workspace(layers, n, DEV)
    P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
    status_ok(ctx)
    # every column of every layer has unit norm (sampled layers: smallest, largest, first, last)
    pick = sorted({0, L - 1, int(np.argmin(sizes)), int(np.argmax(sizes)), L // 2})
    for l in pick:
        blk = W[:, layers[l]:layers[l + 1]].double()
        assert torch.max(torch.abs((blk * blk).sum(dim=1) - 1.0)).item() <= TOL
    g = wl.gradient(0, DEV)
    g_host = g.float().cpu().numpy().astype(np.float64)
    for bits in bits_list:
        lb = twa.twa_quantize_affine(ctx, P32, layers, bits, lws)
        status_ok(ctx)
        packed, a_g, b_g = twa.twa_layered_export(ctx, lb)
        a_h, b_h = a_g.cpu().numpy(), b_g.cpu().numpy()
        cols = [0, n // 2, n - 1]
        for l in pick:
            r0, r1 = layers[l], layers[l + 1]
            blk = np.asfortranarray(W[:, r0:r1].cpu().numpy().T)
            a_o, b_o = orc.affine_factors(blk, [0, r1 - r0], bits)
            assert (a_h[l], b_h[l]) == (a_o[0], b_o[0])
            codes_o = orc.affine_encode(np.asfortranarray(blk[:, cols]), [0, r1 - r0], a_o, b_o, bits)
            lo = r0 - (r0 % 2)
            got = _unpack_rows(packed, lo, r1, bits)[r0 - lo:, :]
            np.testing.assert_array_equal(got[:, cols], codes_o)
        # one step from beta = 0
        sws = twa.new_layered_step_workspace(lb)
        beta = torch.zeros((L, n), device=DEV)
        c = torch.empty((L, n), device=DEV)
        w = torch.empty(D, device=DEV)
        twa.twa_layered_step(ctx, lb, g, LR, 0.0, beta, wbar, w, sws, c_out=c)
        status_ok(ctx)
        c_h, beta_h = c.cpu().numpy(), beta.cpu().numpy()
        np.testing.assert_allclose(beta_h, -LR * c_h.astype(np.float64), rtol=1e-6, atol=1e-30)
        for l in pick:
            r0, r1 = layers[l], layers[l + 1]
            lo = r0 - (r0 % 2)
            codes = _unpack_rows(packed, lo, r1, bits)[r0 - lo:, :][:, cols]
            c_o = orc.project_layerwise(codes, [0, r1 - r0], a_h[l:l + 1], b_h[l:l + 1], g_host[r0:r1])
            scale = abs(float(a_h[l])) * (codes.astype(np.float64).T @ np.abs(g_host[r0:r1])) \
                + abs(float(b_h[l])) * np.abs(g_host[r0:r1]).sum()
            assert np.all(np.abs(c_h[l, cols] - c_o[0]) <= 2e-6 * scale + 1e-30)
        # rows of the lifted weights inside each sampled layer (its first, a middle and its last rows):
        # with the base point, then the lift alone, whose bound is not carried by w_bar
        for base in (wbar, None):
            if base is None:
                twa.twa_layered_lift(ctx, lb, beta, None, w, sws)
                status_ok(ctx)
            for l in pick:
                r0, r1 = layers[l], layers[l + 1]
                span = min(r1 - r0, 3001)
                for s0 in sorted({r0, r0 + (r1 - r0 - span) // 2, r1 - span}):
                    lo = s0 - (s0 % 2)
                    rows_codes = _unpack_rows(packed, lo, s0 + span, bits)[s0 - lo:, :]
                    w_o = orc.lift_layerwise(rows_codes, [0, span], a_h[l:l + 1], b_h[l:l + 1], beta_h[l:l + 1],
                                             None if base is None else base[s0:s0 + span].cpu().numpy())
                    assert rel(w[s0:s0 + span].cpu().numpy(), w_o) <= TOL
        # all layers at once, cheaply: sum_l c[l, i] equals the flat projection of column i
        i = n // 2
        col = _unpack_rows(packed, 0, D, bits)[:, i].astype(np.float64) if D <= 30_000_000 else None
        if col is not None:
            total = 0.0
            for l in range(L):
                r0, r1 = layers[l], layers[l + 1]
                total += float(a_h[l]) * np.dot(col[r0:r1], g_host[r0:r1]) + float(b_h[l]) * g_host[r0:r1].sum()
            assert abs(c_h[:, i].astype(np.float64).sum() - total) <= 1e-5 * np.abs(c_h[:, i]).sum()
        del lb, packed, sws
        torch.cuda.empty_cache()


def test_workload_decoder_layerwise_chunked_sampled(env):
    """The paper's default construction at the 1.3 B size, built from row chunks: mean rows, per-layer
    factors and sampled codes bit-exact against the oracle on the float32 vectors of the build's own
    second pass; one layer-wise step checked on sampled layers, columns and rows."""
    ctx, _ = env
    wl = inputs.WORKLOADS["decoder1p3b"]
    D, n, bits = wl.D, wl.n, 8
    layers = inputs.layer_offsets("decoder1p3b")
    L = len(layers) - 1
    sizes = np.diff(layers)
    CH = inputs.CHUNK_ROWS
    # a bias (2048 rows), a 2048 x 2048 matrix, the layer after the embedding, the last layer
    pick = sorted({1, int(np.argmin(sizes)), int(np.where(sizes == 4194304)[0][len(sizes) // 8]), L - 1})
    blocks = {l: np.empty((layers[l + 1] - layers[l], n), dtype=np.float32, order="F") for l in pick}
    first_rows = {}
    lws = twa.new_layered_workspace(layers, n, DEV)
    wbar = torch.empty(D, device=DEV)
    lb = twa.twa_layered_build_begin(ctx, D, n, layers, bits, lws, DEV)
    buf = torch.empty((n, CH), device=DEV)
    qbuf = torch.empty((n, CH), device=DEV)
    for p in range(3):
        for r0 in range(0, D, CH):
            rows = min(CH, D - r0)
            inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, DEV, row0=r0, rows=rows, out=buf[:, :rows])
            hit = [l for l in pick if layers[l] < r0 + rows and layers[l + 1] > r0] if p == 1 else []
            twa.twa_layered_build_feed(ctx, lb, p, buf, r0, rows, wbar, lws, q32_out=qbuf if hit else None)
            for l in hit:
                a0, a1 = max(layers[l], r0), min(layers[l + 1], r0 + rows)
                blocks[l][a0 - layers[l]:a1 - layers[l]] = qbuf[:, a0 - r0:a1 - r0].cpu().numpy().T
            if p == 0 and r0 in (0, (D // CH) * CH):
                first_rows[r0] = buf[:, :min(rows, 100000)].cpu().numpy().T.copy()
        twa.twa_layered_build_end_pass(ctx, lb, p, lws)
    status_ok(ctx)
    del buf, qbuf
    torch.cuda.empty_cache()
    for r0, a_rows in first_rows.items():
        np.testing.assert_array_equal(wbar[r0:r0 + a_rows.shape[0]].cpu().numpy(), orc.mean(a_rows).astype(np.float32))
    packed, a_g, b_g = twa.twa_layered_export(ctx, lb)
    a_h, b_h = a_g.cpu().numpy(), b_g.cpu().numpy()
    cols = [0, n // 2, n - 1]
    for l in pick:
        r0, r1 = layers[l], layers[l + 1]
        blk = blocks[l]
        # unit columns per layer, factors and codes of the oracle's quantiser on these float32 values
        assert np.max(np.abs(np.sum(blk.astype(np.float64) ** 2, axis=0) - 1.0)) <= TOL
        a_o, b_o = orc.affine_factors(blk, [0, r1 - r0], bits)
        assert (a_h[l], b_h[l]) == (a_o[0], b_o[0])
        codes_o = orc.affine_encode(np.asfortranarray(blk[:, cols]), [0, r1 - r0], a_o, b_o, bits)
        np.testing.assert_array_equal(_unpack_rows(packed, r0, r1, bits)[:, cols], codes_o)
    blocks.clear()
    # one step from beta = 0
    g = wl.gradient(0, DEV)
    sws = twa.new_layered_step_workspace(lb)
    beta = torch.zeros((L, n), device=DEV)
    c = torch.empty((L, n), device=DEV)
    w = torch.empty(D, device=DEV)
    twa.twa_layered_step(ctx, lb, g, LR, 0.0, beta, wbar, w, sws, c_out=c)
    status_ok(ctx)
    c_h, beta_h = c.cpu().numpy(), beta.cpu().numpy()
    np.testing.assert_allclose(beta_h, -LR * c_h.astype(np.float64), rtol=1e-6, atol=1e-30)
    for l in pick:
        r0, r1 = layers[l], layers[l + 1]
        g_l = g[r0:r1].float().cpu().numpy().astype(np.float64)
        codes = _unpack_rows(packed, r0, r1, bits)[:, cols]
        c_o = orc.project_layerwise(codes, [0, r1 - r0], a_h[l:l + 1], b_h[l:l + 1], g_l)
        scale = abs(float(a_h[l])) * (codes.astype(np.float64).T @ np.abs(g_l)) + abs(float(b_h[l])) * np.abs(g_l).sum()
        assert np.all(np.abs(c_h[l, cols] - c_o[0]) <= 2e-6 * scale + 1e-30)
    for base in (wbar, None):
        if base is None:
            twa.twa_layered_lift(ctx, lb, beta, None, w, sws)
            status_ok(ctx)
        for l in pick:
            r0, r1 = layers[l], layers[l + 1]
            span = min(r1 - r0, 3001)
            for s0 in sorted({r0, r0 + (r1 - r0 - span) // 2, r1 - span}):
                lo = s0 - (s0 % 2)
                rows_codes = _unpack_rows(packed, lo, s0 + span, bits)[s0 - lo:, :]
                w_o = orc.lift_layerwise(rows_codes, [0, span], a_h[l:l + 1], b_h[l:l + 1], beta_h[l:l + 1],
                                         None if base is None else base[s0:s0 + span].cpu().numpy())
                assert rel(w[s0:s0 + span].cpu().numpy(), w_o) <= TOL
