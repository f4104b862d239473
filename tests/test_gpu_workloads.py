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
from oracle_stream import HostColumns, WeightedGradientSum, project_f32_columns, project_packed
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
    _PINNED.clear()
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


_PINNED = {}


def to_host(t):
    """A device tensor's bytes as a numpy array, through one reused pinned staging buffer (pageable
    copies of the 10 GB column blocks of the largest workload run at about 2 GB/s)."""
    flat = t.contiguous().view(torch.uint8).reshape(-1)
    buf = _PINNED.get("buf")
    if buf is None or buf.numel() < flat.numel():
        _PINNED["buf"] = None
        buf = torch.empty(flat.numel(), dtype=torch.uint8).pin_memory()
        _PINNED["buf"] = buf
    buf[:flat.numel()].copy_(flat)
    torch.cuda.synchronize()
    return buf[:flat.numel()].numpy().view(np.uint8).reshape(t.shape)


def need_memory(device_gb, host_gb):
    """Skips a test on a box that cannot hold it: free device memory and available host memory in GB."""
    import gc
    import psutil
    gc.collect()
    torch.cuda.empty_cache()                 # what earlier tests freed is still held by the caching allocator
    free, _ = torch.cuda.mem_get_info(0)
    if free < device_gb * 1e9:
        pytest.skip(f"{free / 1e9:.0f} GB free on the device, {device_gb} GB needed")
    avail = psutil.virtual_memory().available
    if avail < host_gb * 1e9:
        pytest.skip(f"{avail / 1e9:.0f} GB of host memory available, {host_gb} GB needed")


def oracle_project_all(ctx, basis, gs, block=8, first_only_blocks=None):
    """The oracle's projection of ALL n columns at full size, for every gradient of the list gs in
    one pass: the canonical codes leave the device eight columns at a time and go through
    oracle.project in row chunks (tests/oracle_stream.py); a float32 basis goes through
    oracle.project_f32 the same way.  Returns C (n, len(gs)) and, per column, a lower bound of
    ||p~_j||: |s_j| qmax (the element that set the scale has the code +-qmax), or for float32 the
    largest |entry|.  With first_only_blocks (a list of block starts) the first gradient of gs is projected
    only on those column blocks (NaN elsewhere): the 1.3 B-sized workload, where a column costs 1.3 G
    multiply-adds on the host."""
    D, n, bits = basis.D, basis.n, basis.bits
    cs, low = [], []
    for j0 in range(0, n, block):
        cols = min(block, n - j0)
        skip_first = first_only_blocks is not None and j0 not in first_only_blocks
        if bits == 32:
            vals = np.asfortranarray(np.stack([basis.data[j, :D].cpu().numpy() for j in range(j0, j0 + cols)], axis=1))
            cs.append(project_f32_columns(vals, gs))
            low.append(np.abs(vals).max(axis=0).astype(np.float64))
            continue
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(basis, col0=j0, cols=cols))
        packed = to_host(codes)                              # valid until the next to_host call
        del codes
        s_h = s.cpu().numpy()
        if skip_first:
            c = project_packed(packed, s_h, D, bits, gs[1:])
            cs.append(np.concatenate([np.full((cols, 1), np.nan), c], axis=1))
        else:
            cs.append(project_packed(packed, s_h, D, bits, gs))
        low.append(np.abs(s_h.astype(np.float64)) * orc.QMAX[bits])
        del packed
    return np.concatenate(cs, axis=0), np.concatenate(low)


def assert_coefficients(c_got, c_ref, norm_low, g_norm):
    """Every one of the n coefficients against the oracle: the stated relative L2 bound, and element
    by element (a single wrong column cannot hide under the norm) 1e-5 of the largest coefficient
    and 1e-5 ||p~_j|| ||g|| with ||p~_j|| replaced by a lower bound of it."""
    c_got = np.asarray(c_got, dtype=np.float64)
    assert rel(c_got, c_ref) <= TOL
    err = np.abs(c_got - c_ref)
    assert np.all(err <= TOL * np.max(np.abs(c_ref)))
    assert np.all(err <= TOL * norm_low * g_norm)


def check_lift_rows(ctx, Pq, bits, w, alpha64, wbar, row_ranges, offset=None):
    """Rows of w against the oracle's lift with the given float64 coefficients: relative L2 and,
    with a base point, a few float32 ulps element by element.  w is the device vector, or (with
    `offset`) a host copy of the rows from `offset` on."""
    D = Pq.D
    seg = 512 * 8 // bits
    for r0, rows in row_ranges:
        assert r0 % seg == 0
        rows = min(rows, D - r0)
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=r0, rows=rows))
        co = orc.unpack_codes(codes.cpu().numpy(), rows, bits)
        base = None if wbar is None else wbar[r0:r0 + rows].cpu().numpy()
        w_ref = orc.lift(co, s.cpu().numpy(), alpha64, base)
        w_got = w[r0:r0 + rows].cpu().numpy() if offset is None else w[r0 - offset:r0 - offset + rows]
        assert rel(w_got, w_ref) <= TOL
        if wbar is not None:
            assert np.max(np.abs(w_got - w_ref.astype(np.float32))) <= 4 * np.spacing(np.float32(np.abs(w_ref).max()))


def sampled_row_ranges(D, bits, n):
    """Row ranges of the lift to compare: the first tiles, the tiles where the second and a middle
    sweep of the persistent grid begin, a range across every multiple of 2^30 rows (the slab boundaries of
    a basis of 2^31 rows or more), the middle, the
    last whole tile and the ragged end.  All start on a 512-byte segment of the codes."""
    seg = 512 * 8 // bits
    tile = seg * (2 if n <= 64 else 1)
    last = ((D - 1) // seg) * seg
    out = [(0, 2 * tile + seg), ((D // 2 // seg) * seg, 3 * seg), (max(0, last - 2 * tile), 2 * tile), (last, seg)]
    for t in (148, 148 * 37 + 5):
        if (t + 2) * tile < D:
            out.append((t * tile - seg, 2 * tile))
    for k in range(1, (D >> 30) + 1):                   # 2^30 and, from 2^31 rows on, every slab boundary
        if D > (k << 30) + 2 * tile:
            out.append(((k << 30) - tile, 2 * tile))
    return sorted(set(out))


def host_columns(ctx, basis, cols):
    """The given columns of a basis on the host for the step-by-step oracle (cols None = all)."""
    D, n = basis.D, basis.n
    cols = list(range(n)) if cols is None else list(cols)
    if not cols:
        return None, cols
    if basis.bits == 32:
        vals = np.asfortranarray(np.stack([basis.data[j, :D].cpu().numpy() for j in cols], axis=1))
        return HostColumns(vals, None, 32), cols
    vals, scales = [], []
    for j in cols:
        codes, s = twa.twa_basis_export(ctx, twa.basis_view(basis, col0=j - j % 8, cols=min(8, n - (j - j % 8))))
        vals.append(orc.unpack_codes(codes[j % 8:j % 8 + 1].cpu().numpy(), D, basis.bits)[:, 0])
        scales.append(s[j % 8].item())
        del codes
    return HostColumns(np.asfortranarray(np.stack(vals, axis=1)), np.array(scales, dtype=np.float32), basis.bits), cols


def run_sequence(ctx, ws, wl, bases, wbar, T, sample_cols, step1_blocks=None):
    """T fused steps from alpha = 0 with a fresh gradient every step (the loop of Algorithm 1 as the
    workload states it), on every basis of `bases` side by side, in the launch configuration the
    benchmark times.  Against the oracle:
      * step 1: all n coefficients c and alpha element by element (with step1_blocks: the columns of
        those blocks of eight), rows of w on sampled ranges;
      * every step: the oracle steps the sampled columns (all columns when sample_cols is None, none
        when it is empty) through project + update; the library's alpha on those columns is compared
        on the way;
      * after step T: all n coefficients against alpha_T = -lr P~^T G, G the weighted sum of the T
        gradients (the oracle's own stepped columns must agree with it to 1e-9), rows of w against
        the oracle's lift with that alpha_T, and the lift alone without the base point."""
    D, n = wl.D, wl.n
    state = []
    for basis in bases:
        cols_h, cols = host_columns(ctx, basis, sample_cols)
        state.append(dict(basis=basis, alpha=torch.zeros(n, device=DEV), w=torch.empty(D, device=DEV),
                          c=torch.empty(n, device=DEV), cols_h=cols_h, cols=cols, a_or=np.zeros(len(cols))))
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    g = torch.empty(D, dtype=gdt, device=DEV)
    g32 = torch.empty(D, device=DEV) if gdt != torch.float32 else None
    g_pin = torch.empty(D, dtype=torch.float32).pin_memory()
    g_host = g_pin.numpy()
    # The weighted sum of the gradients, an INPUT of the oracle's closing projection, is accumulated in
    # float64 by torch on the device (a host adds 1.3 G float64 numbers in seconds, and would do so fifty
    # times over); the same sum is accumulated on the host for sampled row ranges and must agree bit for bit.
    need_host_g = any(len(st["cols"]) for st in state)
    G_dev = torch.zeros(D, dtype=torch.float64, device=DEV)
    span = min(D, 1 << 18)
    sample_rows = sorted({0, ((D // 2) // 4) * 4, D - span})
    gsum = [WeightedGradientSum(span, T, LR, 0.0) for _ in sample_rows]
    g0 = None
    for t in range(T):
        wl.gradient(t, DEV, out=g)
        for st in state:
            twa.twa_step(ctx, st["basis"], g, LR, 0.0, st["alpha"], wbar, st["w"], ws, c_out=st["c"])
        torch.add(G_dev, g, alpha=(1.0 - LR * 0.0) ** (T - 1 - t), out=G_dev)       # widened to float64 by the add
        for r0, acc in zip(sample_rows, gsum):
            acc.add(g[r0:r0 + span].float().cpu().numpy())
        if need_host_g or t == 0:
            if g32 is not None:
                g32.copy_(g)                               # exact widening of bfloat16
            g_pin.copy_(g if g32 is None else g32)
            torch.cuda.synchronize()
        for st in state:
            if len(st["cols"]):
                c_or = st["cols_h"].project(g_host)
                st["a_or"] = orc.sgd_update(st["a_or"], c_or, LR, 0.0)
        if t == 0:
            g0 = g_host.copy()
            for st in state:
                bits = st["basis"].bits
                st["c0"], st["a0"] = st["c"].cpu().numpy(), st["alpha"].cpu().numpy()
                if bits != 32:
                    st["ranges"] = sampled_row_ranges(D, bits, n)
                    st["w0"] = [st["w"][r0:r0 + rows].cpu().numpy() for r0, rows in st["ranges"]]
        if t in (0, T // 3, (2 * T) // 3, T - 1):
            for st in state:
                if len(st["cols"]):
                    assert rel(st["alpha"].cpu().numpy()[st["cols"]], st["a_or"]) <= TOL
    status_ok(ctx)
    del g32
    G = G_dev.cpu().numpy()
    del G_dev
    for r0, acc in zip(sample_rows, gsum):
        np.testing.assert_array_equal(G[r0:r0 + span], acc.result())
    g0_norm = float(np.sqrt(np.dot(g0.astype(np.float64), g0.astype(np.float64))))
    for st in state:
        basis, bits = st["basis"], st["basis"].bits
        a_T = st["alpha"].cpu().numpy()
        C, norm_low = oracle_project_all(ctx, basis, [g0, G], first_only_blocks=step1_blocks)
        c0_ref, a_lin = C[:, 0], -LR * C[:, 1]
        seen = ~np.isnan(c0_ref)                            # columns whose first-step coefficient the oracle computed
        assert seen.sum() >= min(n, 8)
        assert_coefficients(st["c0"][seen], c0_ref[seen], norm_low[seen], g0_norm)
        a0_ref = orc.sgd_update(np.zeros(n), c0_ref, LR, 0.0)
        st["c0_ref"] = c0_ref
        assert_coefficients(st["a0"][seen], a0_ref[seen], LR * norm_low[seen], g0_norm)
        # the lift of step 1 is compared with the oracle's lift of the library's own alpha where the oracle
        # did not project every column (alpha itself is checked on the sampled columns above)
        a0_lift = a0_ref if seen.all() else st["a0"].astype(np.float64)
        if len(st["cols"]):
            assert rel(st["a_or"], a_lin[st["cols"]]) <= 1e-9   # the oracle with itself: stepped = linear form
        assert rel(a_T, a_lin) <= TOL
        assert np.all(np.abs(a_T - a_lin) <= TOL * np.max(np.abs(a_lin)))
        st["a_lin"] = a_lin
        if bits == 32:
            continue                                        # the caller compares the whole of w
        for (r0, rows), w_got in zip(st["ranges"], st["w0"]):
            check_lift_rows(ctx, basis, bits, w_got, a0_lift, wbar, [(r0, rows)], offset=r0)
        check_lift_rows(ctx, basis, bits, st["w"], a_lin, wbar, st["ranges"])
        # the lift alone, without the base point: the bound that is not carried by w_bar
        twa.twa_lift(ctx, basis, st["alpha"], None, st["w"], ws)
        check_lift_rows(ctx, basis, bits, st["w"], a_T.astype(np.float64), None, st["ranges"][:3])
        status_ok(ctx)
    return state


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
    # the workload's 100 steps with a fresh gradient each, float32 and int8 basis side by side; the
    # oracle steps every column; after the last step the whole of w, element by element
    state = run_sequence(ctx, ws, wl, [P32, Pq], wbar, wl.steps, [0, 7, n - 1])
    wbar_h = wbar.cpu().numpy()
    for st, w_o in ((state[0], orc.lift_f32(Pg, state[0]["a_lin"], wbar_h)),
                    (state[1], orc.lift(codes_o, s_o, state[1]["a_lin"], wbar_h))):
        w_g = st["w"].cpu().numpy() if st["basis"].bits == 32 else None
        if w_g is None:                                   # run_sequence ended the int8 leg with a lift without base
            twa.twa_lift(ctx, Pq, st["alpha"], wbar, st["w"], ws)
            w_g = st["w"].cpu().numpy()
        assert rel(w_g, w_o) <= TOL
        assert np.max(np.abs(w_g - w_o.astype(np.float32))) <= 4 * np.spacing(np.float32(np.abs(w_o).max()))
    status_ok(ctx)


# ------------------------------------------------------------------ ResNet-50- and ViT-B-sized: sampled
@pytest.mark.parametrize("name,bits_list", [("resnet50", (8,)), ("vitb16", (8, 4))])
def test_workload_resident_build_sampled(env, name, bits_list):
    """Mean, basis and codes at full size.  The ResNet-50-sized case builds and quantises with the two
    separate calls, the ViT-B/16-sized one with twa_build_quantized (maxima taken during the build):
    everything below is checked against the oracle in both."""
    ctx, ws = env
    wl = inputs.WORKLOADS[name]
    D, n = wl.D, wl.n
    W = wl.candidates(DEV)
    wbar = torch.empty(D, device=DEV)
    one_call = len(bits_list) > 1
    if one_call:
        P32, fused = twa.twa_build_quantized(ctx, W, D, wbar, list(bits_list), ws)
    else:
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
    bases = []
    for k, bits in enumerate(bits_list):
        Pq = fused[k] if one_call else twa.twa_quantize_basis(ctx, P32, bits, ws)
        status_ok(ctx)
        check_codes_sampled(ctx, P32, Pq, bits, [0, n // 2 + 1, n - 1])
        bases.append(Pq)
    del P32, W
    torch.cuda.empty_cache()
    # the workload's 100 steps; the oracle steps two sampled columns
    run_sequence(ctx, ws, wl, bases, wbar, wl.steps, [17, n - 1])
    if name == "vitb16":
        check_batched_projection(ctx, ws, wl, bases)
    del bases
    torch.cuda.empty_cache()


def check_batched_projection(ctx, ws, wl, bases):
    """Eight gradients per projection at full size, in the shape the benchmark times: all n coefficients of
    the group's first and last gradient against the oracle (streamed through the host), and every
    gradient's coefficients against the single projection of the same bytes."""
    D, n = wl.D, wl.n
    batch = 8
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    G = torch.zeros((batch, inputs.padded_ld(D, 8)), dtype=gdt, device=DEV)
    for b in range(batch):
        wl.gradient(1000 + b, DEV, out=G[b, :D])
    g_first = G[0, :D].float().cpu().numpy()
    g_last = G[batch - 1, :D].float().cpu().numpy()
    norms = [float(np.sqrt(np.dot(x.astype(np.float64), x.astype(np.float64)))) for x in (g_first, g_last)]
    for basis in bases:
        assert twa.twa_project_batch_group(ctx, basis, gdt) == batch
        C = torch.empty((batch, n), device=DEV)
        twa.twa_project_batch(ctx, basis, G, C, ws)
        status_ok(ctx)
        C_h = C.cpu().numpy()
        C_or, norm_low = oracle_project_all(ctx, basis, [g_first, g_last])
        assert_coefficients(C_h[0], C_or[:, 0], norm_low, norms[0])
        assert_coefficients(C_h[batch - 1], C_or[:, 1], norm_low, norms[1])
        c = torch.empty(n, device=DEV)
        for b in range(batch):
            twa.twa_project(ctx, basis, G[b, :D], c, ws)
            single = c.cpu().numpy().astype(np.float64)
            assert rel(C_h[b], single) <= 2e-6
            assert np.all(np.abs(C_h[b] - single) <= 2e-6 * np.max(np.abs(single)))
        status_ok(ctx)


# ------------------------------------------------------------------ 1.3 B-sized: chunked build, sampled
def test_workload_decoder_chunked_build_sampled(env):
    """The 1.3 B-sized workload: one row-chunked build gives the int8 and the int4 basis (the scales
    of both widths come from the absmax of pass 2, the codes of both from one feed of pass 3 per chunk);
    then the workload's 50 steps on both, checked as run_sequence describes."""
    ctx, ws = env
    wl = inputs.WORKLOADS["decoder1p3b"]
    D, n = wl.D, wl.n
    CH = inputs.CHUNK_ROWS
    starts = list(range(0, D, CH))
    sampled = {starts[0]: None, starts[len(starts) // 2]: None, starts[-1]: None}
    bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=DEV)
    wbar = torch.empty(D, device=DEV)
    bases = {bits: twa.new_quantised_basis(D, n, bits, DEV) for bits in (8, 4)}
    buf = torch.empty((n, CH), device=DEV)
    qbuf = torch.empty((n, CH), device=DEV)
    twa.twa_build_begin(ctx, D, n, wbar, bws)
    for p in range(4):
        for r0 in starts:
            rows = min(CH, D - r0)
            inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, DEV, row0=r0, rows=rows, out=buf[:, :rows])
            keep = p == 3 and r0 in sampled
            if p < 3:
                twa.twa_build_feed(ctx, p, buf, r0, rows)
            else:
                twa.twa_build_feed_codes(ctx, buf, r0, rows, [bases[8], bases[4]], q32_out=qbuf if keep else None)
            if keep:
                sampled[r0] = (qbuf[:, :rows].cpu().numpy().T.copy(), buf[:, :rows].cpu().numpy().T.copy())
        if p == 2:
            twa.twa_build_end_pass(ctx, p, 8, bases[8])
            twa.twa_build_end_pass(ctx, p, 4, bases[4])
        else:
            twa.twa_build_end_pass(ctx, p, 0, None)
    status_ok(ctx)
    del buf, qbuf, bws
    torch.cuda.empty_cache()
    for bits, Pq in bases.items():
        scales = Pq.scales.cpu().numpy()
        qmax = orc.QMAX[bits]
        for r0, (q32, a_rows) in sampled.items():
            rows = q32.shape[0]
            # codes of the chunk = the oracle's encoder on the chunk's float32 rows with the global scales
            codes, _ = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=r0, rows=rows))
            co = orc.encode(np.asfortranarray(q32), scales, bits)
            np.testing.assert_array_equal(codes.cpu().numpy(), orc.pack_codes(co, bits))
            assert np.all(np.abs(q32).max(axis=0) <= scales * qmax * (1 + 1e-6))
            del codes, co
    M0 = None
    for r0, (q32, a_rows) in sampled.items():
        rows = q32.shape[0]
        # w_bar rows = the oracle's mean of the candidate rows
        np.testing.assert_array_equal(wbar[r0:r0 + rows].cpu().numpy(), orc.mean(a_rows).astype(np.float32))
        # rows of Q are rows of A times one upper-triangular matrix: the same M for every chunk
        if M0 is None:
            M0, *_ = np.linalg.lstsq(a_rows[:65536].astype(np.float64), q32[:65536].astype(np.float64), rcond=None)
            assert np.max(np.abs(np.tril(M0, -1))) <= 1e-3 * np.max(np.abs(M0))
            assert np.all(np.diag(M0) > 0)
        else:
            resid = a_rows[:65536].astype(np.float64) @ M0 - q32[:65536]
            assert np.linalg.norm(resid) <= 1e-5 * np.linalg.norm(q32[:65536])
    sampled.clear()
    # unit columns: the dequantised basis has norm 1 up to the quantisation error (oracle on one column)
    codes, s = twa.twa_basis_export(ctx, twa.basis_view(bases[8], col0=24, cols=8))
    col = codes[7].cpu().numpy().view(np.int8)[:D].astype(np.float64)
    assert abs(np.sqrt(np.dot(col, col)) * float(s[7]) - 1.0) <= 2e-3
    del codes, col
    torch.cuda.empty_cache()
    run_sequence(ctx, ws, wl, [bases[8], bases[4]], wbar, wl.steps, [], step1_blocks=[0, 24])


def test_basis_of_more_than_2_31_rows(env):
    """A basis of 2^31 + 3 * 2^22 + 70,001 rows (three slabs of the stepping calls; odd, so the 4-bit
    column ends on a half byte) and four columns: row-chunked build of the int8 and the int4 basis,
    mean, codes and scales of sampled chunks (the first, the one that ends at row 2^31, the last)
    against the oracle, then two fused steps on both widths checked as run_sequence describes: all
    coefficients after step 1 and step 2, rows of w at the start, across 2^30, across 2^31, in the
    last slab and at the ragged end."""
    ctx, ws = env
    need_memory(100, 80)
    D, n = (1 << 31) + 3 * (1 << 22) + 70_001, 4
    wl = inputs.Workload("rows_2g", D, n, 0.002, 0.0005, 1e-4, "bf16", (8, 4), 2, seed=11, chunked_build=True)
    CH = inputs.CHUNK_ROWS
    starts = list(range(0, D, CH))
    sampled = {starts[0]: None, (1 << 31) - CH: None, starts[-1]: None}
    bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=DEV)
    wbar = torch.empty(D, device=DEV)
    bases = {bits: twa.new_quantised_basis(D, n, bits, DEV) for bits in (8, 4)}
    buf = torch.empty((n, CH), device=DEV)
    qbuf = torch.empty((n, CH), device=DEV)
    twa.twa_build_begin(ctx, D, n, wbar, bws)
    for p in range(4):
        for r0 in starts:
            rows = min(CH, D - r0)
            inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, DEV, row0=r0, rows=rows, out=buf[:, :rows])
            keep = p == 3 and r0 in sampled
            if p < 3:
                twa.twa_build_feed(ctx, p, buf, r0, rows)
            else:
                twa.twa_build_feed_codes(ctx, buf, r0, rows, [bases[8], bases[4]], q32_out=qbuf if keep else None)
            if keep:
                sampled[r0] = (qbuf[:, :rows].cpu().numpy().T.copy(), buf[:, :rows].cpu().numpy().T.copy())
        if p == 2:
            twa.twa_build_end_pass(ctx, p, 8, bases[8])
            twa.twa_build_end_pass(ctx, p, 4, bases[4])
        else:
            twa.twa_build_end_pass(ctx, p, 0, None)
    status_ok(ctx)
    del buf, qbuf, bws
    torch.cuda.empty_cache()
    M0 = None
    for r0, (q32, a_rows) in sampled.items():
        rows = q32.shape[0]
        np.testing.assert_array_equal(wbar[r0:r0 + rows].cpu().numpy(), orc.mean(a_rows).astype(np.float32))
        for bits, Pq in bases.items():
            scales = Pq.scales.cpu().numpy()
            codes, _ = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=r0, rows=rows))
            co = orc.encode(np.asfortranarray(q32), scales, bits)
            np.testing.assert_array_equal(codes.cpu().numpy(), orc.pack_codes(co, bits))
            assert np.all(np.abs(q32).max(axis=0) <= scales * orc.QMAX[bits] * (1 + 1e-6))
            del codes, co
        # rows of Q are rows of A times one upper-triangular matrix with a positive diagonal: the same for every chunk
        if M0 is None:
            M0, *_ = np.linalg.lstsq(a_rows[:65536].astype(np.float64), q32[:65536].astype(np.float64), rcond=None)
            assert np.max(np.abs(np.tril(M0, -1))) <= 1e-3 * np.max(np.abs(M0))
            assert np.all(np.diag(M0) > 0)
        else:
            resid = a_rows[:65536].astype(np.float64) @ M0 - q32[:65536]
            assert np.linalg.norm(resid) <= 1e-5 * np.linalg.norm(q32[:65536])
    sampled.clear()
    # unit columns: the dequantised int8 column has norm 1 up to the quantisation error (whole-basis export)
    codes, s = twa.twa_basis_export(ctx, bases[8])
    col = codes[n - 1].cpu().numpy().view(np.int8)[:D]
    sq = sum(float(np.dot(col[a:a + (1 << 26)].astype(np.float64), col[a:a + (1 << 26)].astype(np.float64)))
             for a in range(0, D, 1 << 26))
    assert abs(np.sqrt(sq) * float(s[n - 1]) - 1.0) <= 2e-3
    del codes, col
    torch.cuda.empty_cache()
    state = run_sequence(ctx, ws, wl, [bases[8], bases[4]], wbar, wl.steps, [])
    # the Adam step over the slabs: first step from zero moments on the first gradient, against the oracle's
    # Adam update of the oracle's own coefficients' gradient
    g = wl.gradient(0, DEV)
    for st in state:
        alpha, m, v = (torch.zeros(n, device=DEV) for _ in range(3))
        w = st["w"]
        twa.twa_step_adam(ctx, st["basis"], g, 1e-2, 1, alpha, m, v, wbar, w, ws, weight_decay=0.01)
        a_ref, m_ref, v_ref = orc.adam_update(np.zeros(n), np.zeros(n), np.zeros(n), st["c0_ref"], 1e-2, 1,
                                              weight_decay=0.01)
        assert rel(m.cpu().numpy(), m_ref) <= TOL and rel(v.cpu().numpy(), v_ref) <= 2 * TOL
        assert rel(alpha.cpu().numpy(), a_ref) <= TOL
        check_lift_rows(ctx, st["basis"], st["basis"].bits, w, a_ref, wbar, st["ranges"][-3:])
    # the step from host memory (sixteen row chunks, not the three slabs): same alpha to rounding, same rows of w
    st = state[0]
    g_host = torch.empty(D, dtype=torch.bfloat16).pin_memory()
    g_host.copy_(g)
    w_host = torch.empty(D, dtype=torch.float32).pin_memory()
    g_stage = torch.empty(D, dtype=torch.bfloat16, device=DEV)
    alpha = torch.zeros(n, device=DEV)
    twa.twa_step_host(ctx, st["basis"], g_host, LR, 0.0, alpha, wbar, st["w"], w_host, g_stage, ws)
    status_ok(ctx)
    a0_ref = orc.sgd_update(np.zeros(n), st["c0_ref"], LR, 0.0)
    assert rel(alpha.cpu().numpy(), a0_ref) <= TOL
    check_lift_rows(ctx, st["basis"], 8, st["w"], a0_ref, wbar, st["ranges"])
    for r0, rows in st["ranges"]:
        np.testing.assert_array_equal(w_host[r0:r0 + rows].numpy(), st["w"][r0:r0 + rows].cpu().numpy())
    del g_host, w_host, g_stage
    # the calls whose kernels index rows with 32-bit integers refuse the whole basis and take a view of it
    c = torch.empty(n, device=DEV)
    with pytest.raises(twa.TwaError):
        twa.twa_project_noalloc(0, None, bases[8], torch.zeros(D, dtype=torch.bfloat16, device=DEV), c)


@pytest.mark.parametrize("D", [(1 << 31) - 5, (1 << 31) + 70_001])
def test_float32_candidates_of_more_than_2_31_rows(env, D):
    """Two float32 candidates of 2^31 - 5 rows (above the row count one launch takes, so two slabs whose
    second is five rows short of 2^30) and of 2^31 + 70,001 rows: the fixed-weight average (the float32 lift over the
    slabs) on rows at the start, across 2^30 and 2^31 and at the end against the oracle, and the float32
    projection on all rows against the oracle's, streamed through the host, on integer-valued inputs
    that make the result exact."""
    ctx, ws = env
    need_memory(60, 40)
    n = 2
    wl = inputs.Workload("rows_2g_f32", D, n, 0.002, 0.0005, 1e-3, "f32", (32,), 1, seed=12)
    W = torch.zeros((n, (D + 3) // 4 * 4), device=DEV)      # columns start on 16 bytes
    CH = inputs.CHUNK_ROWS
    for r0 in range(0, D, CH):
        rows = min(CH, D - r0)
        inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, DEV, row0=r0, rows=rows, out=W[:, r0:r0 + rows])
    weights = torch.tensor([0.25, 0.75], device=DEV)
    w = torch.empty(D, device=DEV)
    twa.twa_weighted_average(ctx, W, D, weights, w, ws)
    status_ok(ctx)
    span = 1 << 16
    for r0 in sorted({0, (1 << 30) - span // 2, min((1 << 31) - span // 2, D - span), D - span}):
        rows_h = W[:, r0:r0 + span].cpu().numpy().T
        ref = orc.weighted_average(rows_h, [0.25, 0.75])
        got = w[r0:r0 + span].cpu().numpy()
        assert rel(got, ref) <= TOL
        assert np.max(np.abs(got - ref.astype(np.float32))) <= 4 * np.spacing(np.float32(np.abs(ref).max()))
    # the float32 projection on small integers (candidates in [-2, 2], gradient in [-1, 1]): every partial
    # sum is an integer below 2^24, so the float32 sums are exact in any order and the oracle's float64
    # result must be met to the last bit, float32 and bfloat16 gradient alike
    inputs.small_integers(W[:, :D], -2, 2, wl.seed)
    g = inputs.small_integers(torch.empty((1, D), device=DEV), -1, 1, wl.seed + 1)[0]
    c = torch.empty(n, device=DEV)
    twa.twa_project(ctx, twa.basis_from_tensor(W, D), g, c, ws)
    status_ok(ctx)
    c16 = torch.empty(n, device=DEV)
    twa.twa_project(ctx, twa.basis_from_tensor(W, D), g.to(torch.bfloat16), c16, ws)
    status_ok(ctx)
    g_h = to_host(g.view(torch.uint8)).view(np.float32).copy()
    c_ref = np.zeros(n)
    for j in range(n):
        col = to_host(W[j, :D].view(torch.uint8)).view(np.float32).reshape(-1, 1)
        c_ref[j] = project_f32_columns(col, [g_h])[0, 0]
    assert np.all(c_ref == np.rint(c_ref)) and np.all(np.abs(c_ref) < 2 ** 24) and np.any(c_ref != 0)
    np.testing.assert_array_equal(c.cpu().numpy().astype(np.float64), c_ref)
    np.testing.assert_array_equal(c16.cpu().numpy().astype(np.float64), c_ref)


# ------------------------------------------------------------------ the layer-wise construction, full size
def _unpack_rows(packed, r0, r1, bits):
    """Unsigned codes of flat rows r0..r1-1 (r0 a multiple of the codes per byte) from the canonical
    export, shape (rows, n), by the oracle's definition of that image."""
    slot = orc.SLOT_BITS[bits]
    assert (r0 * slot) % 8 == 0
    b = packed[:, r0 * slot // 8:(r1 * slot + 7) // 8].cpu().numpy()
    return orc.unpack_unsigned(b, r1 - r0, bits)


@pytest.mark.parametrize("name,bits_list", [("resnet50", (8, 16)), ("vitb16", (8, 4, 3, 2, 1))])
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
            lo = r0 - (r0 % 8)
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
            lo = r0 - (r0 % 8)
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
                    lo = s0 - (s0 % 8)
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


@pytest.mark.parametrize("bits", [8, 4])
def test_workload_decoder_layerwise_chunked_sampled(env, bits):
    """The paper's default construction at the 1.3 B size, built from row chunks: mean rows, per-layer
    factors and codes of sampled layers bit-exact against the oracle on the float32 vectors of the
    build's own second pass; one layer-wise step checked on sampled layers (all n columns) and rows."""
    ctx, _ = env
    wl = inputs.WORKLOADS["decoder1p3b"]
    D, n = wl.D, wl.n
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
    cols = list(range(n))
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
                lo = s0 - (s0 % 8)
                rows_codes = _unpack_rows(packed, lo, s0 + span, bits)[s0 - lo:, :]
                w_o = orc.lift_layerwise(rows_codes, [0, span], a_h[l:l + 1], b_h[l:l + 1], beta_h[l:l + 1],
                                         None if base is None else base[s0:s0 + span].cpu().numpy())
                assert rel(w[s0:s0 + span].cpu().numpy(), w_o) <= TOL
