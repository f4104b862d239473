"""GPU parity for the projection of several gradients at once (two gradients per integer MMA)
against the float64 oracle applied column by column, and against the single-gradient call."""

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


def _basis(ctx, ws, D, n, bits, seed):
    gen = torch.Generator(device=DEV).manual_seed(seed)
    P = torch.zeros((n, inputs.padded_ld(D, 4)), device=DEV)
    P[:, :D] = torch.randn((n, D), generator=gen, device=DEV) / np.sqrt(D)
    P32 = twa.basis_from_tensor(P, D)
    if bits == 32:
        return P32, P
    return twa.twa_quantize_basis(ctx, P32, bits, ws), P


def _gradients(D, batch, dtype, seed):
    ld = inputs.padded_ld(D, 8)
    gen = torch.Generator(device=DEV).manual_seed(seed)
    G = torch.full((batch, ld), float("nan"), device=DEV)          # the padding must never be read
    G[:, :D] = torch.randn((batch, D), generator=gen, device=DEV) * 1e-3
    # rows of very different magnitude: every gradient needs its own digit scale
    G[:, :D] *= (10.0 ** torch.arange(batch, device=DEV).remainder(5))[:, None]
    return G.to(dtype)


@pytest.mark.parametrize("gdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("D,n,batch", [(5, 2, 3), (4099, 33, 8), (70001, 100, 4), (70001, 100, 7), (33333, 128, 9),
                                       (300007, 20, 13), (150001, 64, 16), (2049, 1, 1), (51234, 70, 2)])
def test_project_batch(env, D, n, batch, bits, gdt):
    ctx, ws = env
    Pq, _ = _basis(ctx, ws, D, n, bits, 300 + D + n)
    G = _gradients(D, batch, gdt, D + batch)
    C = torch.full((batch + 1, n), 7.0, device=DEV)
    twa.twa_project_batch(ctx, Pq, G, C[:batch], ws)
    status_ok(ctx)
    codes, s = twa.twa_basis_export(ctx, Pq)
    co = orc.unpack_codes(codes.cpu().numpy(), D, bits)
    C_o = orc.project_batch(co, s.cpu().numpy(), G[:, :D].float().cpu().numpy().T)     # (n, batch)
    C_g = C[:batch].cpu().numpy().T
    for b in range(batch):
        assert rel(C_g[:, b], C_o[:, b]) <= TOL, b
    assert torch.all(C[batch] == 7.0)
    # the single-gradient call gives the same numbers up to its own rounding
    c1 = torch.empty(n, device=DEV)
    for b in (0, batch - 1):
        twa.twa_project(ctx, Pq, G[b, :D], c1, ws)
        assert rel(c1.cpu().numpy(), C_o[:, b]) <= TOL
        assert rel(C_g[:, b], c1.cpu().numpy()) <= 2 * TOL
    # fixed summation order: the same call again is bitwise the same
    C2 = torch.empty((batch, n), device=DEV)
    twa.twa_project_batch(ctx, Pq, G, C2, ws)
    assert torch.equal(C2, C[:batch])


@pytest.mark.parametrize("bits", [8, 4])
def test_project_batch_replayed_from_a_cuda_graph(bits):
    """twa_project_batch (two passes of eight gradients here) captured once and replayed on new bytes
    in the same gradient buffer: the coefficients of a direct call, bit for bit."""
    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    D, n, batch = 70001, 33, 11
    with torch.cuda.stream(stream):
        ctx = twa.twa_create(0, stream=stream)
        ws = twa.new_workspace(DEV)
        B, _ = _basis(ctx, ws, D, n, bits, 5)
        G_buf = torch.zeros_like(_gradients(D, batch, torch.bfloat16, 1))
        C_g = torch.empty((batch, n), device=DEV)
        twa.twa_project_batch(ctx, B, G_buf, C_g, ws)                  # warm-up outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            twa.twa_project_batch(ctx, B, G_buf, C_g, ws)
        for seed in (2, 3):
            G = _gradients(D, batch, torch.bfloat16, seed)
            C_d = torch.empty((batch, n), device=DEV)
            twa.twa_project_batch(ctx, B, G, C_d, ws)
            G_buf.copy_(G)
            graph.replay()
            stream.synchronize()
            assert torch.equal(C_g, C_d)
        status_ok(ctx)
        del graph
        twa.twa_destroy(ctx)


def test_project_batch_float32_basis_and_group(env):
    ctx, ws = env
    D, n, batch = 10007, 6, 3
    P32, P = _basis(ctx, ws, D, n, 32, 9)
    assert twa.twa_project_batch_group(ctx, P32) == 1
    G = _gradients(D, batch, torch.float32, 4)
    C = torch.empty((batch, n), device=DEV)
    twa.twa_project_batch(ctx, P32, G, C, ws)
    status_ok(ctx)
    Ph = P[:, :D].cpu().numpy().T
    for b in range(batch):
        assert rel(C[b].cpu().numpy(), orc.project_f32(Ph, G[b, :D].cpu().numpy())) <= TOL
    Pq, _ = _basis(ctx, ws, D, n, 8, 9)
    assert twa.twa_project_batch_group(ctx, Pq) == 8
    Pw, _ = _basis(ctx, ws, D, 100, 8, 9)
    assert twa.twa_project_batch_group(ctx, Pw) == 8
    assert twa.twa_project_batch_group(ctx, Pw, torch.float32) in (4, 8)


def test_project_batch_zero_and_nonfinite_gradients(env):
    ctx, ws = env
    D, n, batch = 40000, 12, 5
    Pq, _ = _basis(ctx, ws, D, n, 8, 77)
    G = _gradients(D, batch, torch.float32, 5)
    G[1] = 0.0                                   # a gradient of zeros beside a live one in the same MMA
    G[1, D:] = float("nan")
    G[3, 123] = float("inf")
    C = torch.empty((batch, n), device=DEV)
    twa.twa_project_batch(ctx, Pq, G, C, ws)
    code, detail = twa.twa_get_status(ctx)
    assert (code, detail) == (twa.TWA_ERR_NONFINITE, 3)
    twa.twa_clear_status(ctx)
    assert torch.all(C[1] == 0) and torch.isnan(C[3]).all()
    codes, s = twa.twa_basis_export(ctx, Pq)
    co = orc.unpack_codes(codes.cpu().numpy(), D, 8)
    for b in (0, 2, 4):                          # the neighbours of the bad gradient are untouched
        assert rel(C[b].cpu().numpy(), orc.project(co, s.cpu().numpy(), G[b, :D].cpu().numpy())) <= TOL
    # argument checks on the host
    with pytest.raises(twa.TwaError) as e:
        twa.twa_project_batch(ctx, Pq, G[:, 1:].contiguous()[:, : D + 3].contiguous(), C, ws)
    assert e.value.code in (twa.TWA_ERR_MISALIGNED, twa.TWA_ERR_INVALID_ARG)
