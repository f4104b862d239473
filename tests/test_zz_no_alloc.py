"""twa_project_noalloc: the projection for callers that cannot allocate device memory when
they call (an allocator that owns the whole device, a loop that may not synchronise, a
plug-in given only its buffers).  It must give what twa_project gives -- and what the float64
oracle gives on the same bytes -- call after call, although it has no context and no workspace
and keeps its scratch in a fixed array of the library's device image that every call reuses.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""

import numpy as np
import pytest
import torch

from oracle import twa_oracle as orc
from paper_2205_13104_b200 import twa

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-5            # the bound of the projection parity tests


def _rel(x, y):
    x, y = x.double(), y.double()
    return float((x - y).norm() / y.norm())


@pytest.mark.parametrize("bits,gdt", [(8, torch.bfloat16), (4, torch.float32), (32, torch.float32)])
def test_noalloc_projection_matches_twa_project_twice_in_a_row(bits, gdt):
    torch.cuda.set_device(0)
    D, n = 300007, 33
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1234 + bits)
    ld = (D + 3) // 4 * 4
    P = torch.zeros((n, ld), device=DEV)
    P[:, :D] = torch.randn((n, D), generator=gen, device=DEV) / np.sqrt(D)
    ctx = twa.twa_create(0)
    ws = twa.new_workspace(DEV)
    B = twa.basis_from_tensor(P, D)
    if bits != 32:
        B = twa.twa_quantize_basis(ctx, B, bits, ws)
    if bits != 32:                             # the oracle's view of the same basis: canonical codes and scales
        codes, scales = twa.twa_basis_export(ctx, B)
        codes_h, scales_h = orc.unpack_codes(codes.cpu().numpy(), D, bits), scales.cpu().numpy()
    else:
        P_h = P[:, :D].cpu().numpy().T
    status = torch.full((2,), 99, dtype=torch.int32, device=DEV)
    for call in range(2):                      # the second call meets the first one's leftovers
        g = (torch.randn(D, generator=gen, device=DEV) * 1e-3).to(gdt)
        want = torch.empty(n, device=DEV)
        twa.twa_project(ctx, B, g, want, ws)
        got = torch.full((n + 2,), 5.0, device=DEV)
        twa.twa_project_noalloc(0, None, B, g, got, status)
        torch.cuda.synchronize()
        assert status[0].item() == 0
        assert _rel(got[:n], want) <= TOL
        assert torch.all(got[n:] == 5.0)
        g_h = g.float().cpu().numpy()
        c_o = orc.project(codes_h, scales_h, g_h) if bits != 32 else orc.project_f32(P_h, g_h)
        assert _rel(got[:n].cpu(), torch.from_numpy(c_o)) <= TOL
        assert _rel(want.cpu(), torch.from_numpy(c_o)) <= TOL
    assert twa.twa_get_status(ctx)[0] == 0
    twa.twa_destroy(ctx)


def test_noalloc_rejects_what_the_static_scratch_cannot_hold():
    torch.cuda.set_device(0)
    D = 4096
    P = torch.zeros((twa.TWA_MAX_N + 1, D), device=DEV)
    B = twa.basis_from_tensor(P, D)
    g = torch.zeros(D, device=DEV)
    c = torch.zeros(twa.TWA_MAX_N + 1, device=DEV)
    with pytest.raises(twa.TwaError) as e:
        twa.twa_project_noalloc(0, None, B, g, c)
    assert e.value.code == twa.TWA_ERR_UNSUPPORTED
    assert "static scratch" in str(e.value)
    assert twa.twa_noalloc_scratch_bytes() == 256 * 128 * 4 + 256
