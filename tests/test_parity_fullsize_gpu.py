"""Parity at the full benchmark sizes (2D 2048^2 x 16 and 3D 256^3 x 4, and the two mid-size workloads 2D 256^2 x 64 and
3D 64^3 x 32), in the launch configuration the benchmark times: every node of the residual and every sample's energy
against the oracle's full pass, in all three diffusivity modes, plus properties that hold at any size; and the
energy-only call on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, J_RTOL, R_RTOL, guarded, guards_intact

pytestmark = pytest.mark.gpu

PATHS = {1: ("row2d", "tiled2d"), 2: ("strip2d",), 3: ("strip3d",), 4: ("strip3d",)}   # cfg1 with a stored field: tiled2d


@pytest.mark.parametrize("mode", [B.DN_NU_KL_GAUSS, B.DN_NU_NODAL, B.DN_NU_KL_NODAL])
@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_fullsize_every_node(cfg, mode):
    inp = inputs.make_inputs(cfg)
    ud = dev(inp.u)
    wd = dev(inp.kl_w)
    nu_d = None
    if mode == B.DN_NU_NODAL:
        nu_d = torch.empty(inp.u.shape, device="cuda")
        B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, wd, nu_d)
    pg = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu_d,
                   kl_modes=inp.kl_modes, kl_w=wd, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    assert B.dn_path_name(pg) in PATHS[cfg]                            # the kernel family the benchmark times
    n = inp.u.size
    r_whole, r_bytes = guarded(4 * n)
    r = r_bytes.view(torch.float32).view(inp.u.shape)
    r.fill_(float("nan"))
    J = torch.full((inp.batch,), float("nan"), device="cuda")
    ws_n = B.dn_workspace_bytes(pg)
    ws_whole, ws = guarded(ws_n)
    B.dn_energy_grad(pg, ud, None, J, r, ws)
    torch.cuda.synchronize()
    assert guards_intact(r_whole, 4 * n) and guards_intact(ws_whole, ws_n)
    Jg = J.cpu().numpy().astype(np.float64)
    Je = torch.full((inp.batch,), float("nan"), device="cuda")
    B.dn_energy(pg, ud, Je, ws)                                     # the energy-only call: same inputs, same workspace
    Je = Je.cpu().numpy().astype(np.float64)
    nu_h = nu_d.cpu().numpy() if nu_d is not None else None        # the oracle reads the same float32 field
    po = oracle.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu_h,
                        kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    # 1. the oracle's full pass: every sample's energy, every node's residual; the scale is the oracle's own maximum
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    rel = np.abs(Jg - Jo) / np.abs(Jo)
    assert np.all(rel <= J_RTOL), f"J rel err {rel} J*={Jo}"
    assert np.all(np.abs(Je - Jo) <= J_RTOL * np.abs(Jo)), f"dn_energy: J rel err {np.abs(Je - Jo) / np.abs(Jo)}"
    scale = np.abs(ro).max()
    worst = 0.0
    for b in range(inp.batch):                                      # sample by sample: bounded host memory
        rg = r[b].cpu().numpy()
        assert np.isfinite(rg).all()
        worst = max(worst, float(np.abs(rg - ro[b]).max()))
    assert worst <= R_RTOL * scale, f"r max err {worst:.3e} vs max|r*| {scale:.3e} ({worst / scale:.2e})"
    del ro
    # 2. properties at any size: Dirichlet mask, partition of unity of the unmasked residual
    assert float(r[..., 0].abs().max()) == 0.0 and float(r[..., -1].abs().max()) == 0.0
    pg.flags = B.DN_NO_MASK
    B.dn_energy_grad(pg, ud, None, None, r, ws)
    s = r.double().sum(dim=tuple(range(1, r.dim()))).cpu().numpy()
    l1 = r.double().abs().sum(dim=tuple(range(1, r.dim()))).cpu().numpy()
    assert np.all(np.abs(s + inp.f_const) <= 2e-6 * l1 + 1e-6), (s, l1)
