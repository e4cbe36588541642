"""Parity at the full benchmark sizes (2D 2048^2 x 16 and 3D 256^3 x 4), in the launch configuration
the benchmark times: every sample's energy and sampled residual nodes against the oracle, plus
properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, make_problems, J_RTOL, R_RTOL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [B.DN_NU_KL_GAUSS, B.DN_NU_NODAL])
@pytest.mark.parametrize("cfg", [2, 4])
def test_fullsize_sampled(cfg, mode):
    wl = inputs.WORKLOADS[cfg]
    inp = inputs.make_inputs(cfg)
    ud = dev(inp.u)
    wd = dev(inp.kl_w)
    nu_d = None
    if mode == B.DN_NU_NODAL:
        nu_d = torch.empty(inp.u.shape, device="cuda")
        B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, wd, nu_d)
    pg = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu_d,
                   kl_modes=inp.kl_modes, kl_w=wd, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    r = torch.empty(inp.u.shape, device="cuda"); J = torch.empty(inp.batch, device="cuda")
    B.dn_energy_grad(pg, ud, None, J, r, B.new_workspace(pg))
    torch.cuda.synchronize()
    Jg = J.cpu().numpy().astype(np.float64)
    nu_h = nu_d.cpu().numpy() if nu_d is not None else None        # the oracle reads the same float32 field
    po = oracle.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu_h,
                        kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    # 1. sampled nodes: random ones plus the corners / edges / tile seams of the domain
    rng = np.random.default_rng(cfg)
    nodes = wl.nodes
    idx = rng.integers(0, inp.batch * nodes, size=30000)
    n = wl.n
    special = []
    # 124 k .. 124 k + 4: where neighbouring strips of the 2D strip kernel overlap; 128 / 256: warp seams of the tiled kernels
    coords = [0, 1, 2, 3, 4, 123, 124, 127, 128, 129, 247, 248, 251, 252, 255, 256, 371, 372, 375, 376, 1983, 1984, 1987, 1988,
              n // 2 - 1, n // 2, n - 5, n - 4, n - 3, n - 2, n - 1]
    coords = sorted({c for c in coords if 0 <= c < n})
    for b in (0, inp.batch - 1):
        for iy in coords:
            for ix in coords:
                if inp.dim == 2:
                    special.append((b * n + iy) * n + ix)
                else:
                    for iz in coords[::3] + [n - 1]:
                        special.append(((b * n + iz) * n + iy) * n + ix)
    idx = np.unique(np.concatenate([idx, np.array(special, dtype=np.int64)]))
    ro = oracle.residual_at(po, inp.u, idx)
    rg = r.view(-1)[torch.from_numpy(idx).cuda()].cpu().numpy().astype(np.float64)
    scale = float(r.abs().max())
    assert np.isfinite(rg).all()
    err = np.abs(rg - ro).max()
    assert err <= R_RTOL * max(scale, np.abs(ro).max()), f"sampled r err {err:.3e} vs scale {scale:.3e}"
    # 2. the energy of every sample (the oracle's full pass, energy only)
    Jo = oracle.energy_grad(po, inp.u, want_r=False)[0]
    rel = np.abs(Jg - Jo) / np.abs(Jo)
    assert np.all(rel <= J_RTOL), f"J rel err {rel} J*={Jo}"
    # 3. properties at any size: Dirichlet mask, partition of unity of the unmasked residual
    assert float(r[..., 0].abs().max()) == 0.0 and float(r[..., -1].abs().max()) == 0.0
    pg.flags = B.DN_NO_MASK
    B.dn_energy_grad(pg, ud, None, None, r, B.new_workspace(pg))
    s = r.double().sum(dim=tuple(range(1, r.dim()))).cpu().numpy()
    l1 = r.double().abs().sum(dim=tuple(range(1, r.dim()))).cpu().numpy()
    assert np.all(np.abs(s + inp.f_const) <= 2e-6 * l1 + 1e-6), (s, l1)
