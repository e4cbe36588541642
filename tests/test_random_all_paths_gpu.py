"""Seeded random problems across every kernel family (2D and 3D, narrow and wide rows, all diffusivity modes, both kinds
of forcing, every flag): the fused call and the energy-only call against the oracle.  Whatever family the shape selects
is the one under test; the last test checks that the seeds reach all of them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, make_problems, run_gpu, check, guarded, guards_intact

pytestmark = pytest.mark.gpu

MODES = [B.DN_NU_KL_GAUSS, B.DN_NU_KL_NODAL, B.DN_NU_NODAL]
N_CASES = 96


def draw(i):
    rng = np.random.default_rng(100000 + i)
    dim = int(rng.choice([2, 3]))
    if dim == 2:
        narrow = rng.random() < 0.5
        nx = int(rng.choice([8, 12, 16, 20, 28, 36, 64, 96, 100, 128, 132, 136, 192, 248, 256])) if narrow else 4 * int(rng.integers(65, 640))
        ny, nz, batch = int(rng.integers(2, 120)), 1, int(rng.integers(1, 12))
    else:
        nx = int(rng.choice([8, 12, 16, 24, 32, 36, 48, 64, 72, 100, 128, 136, 192, 256, 260, 300]))
        ny, nz, batch = int(rng.integers(2, 20)), int(rng.integers(2, 20)), int(rng.integers(1, 5))
    m, mode = int(rng.integers(1, 9)), MODES[int(rng.integers(0, 3))]
    flags = int(rng.choice([0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK]))
    f_const = float(rng.choice([0.0, 0.7]))
    nodal_f, with_gJ = rng.random() < 0.35, rng.random() < 0.5
    gJ = rng.uniform(-2, 2, batch).astype(np.float32) if with_gJ else None
    return dim, nx, ny, nz, batch, m, mode, flags, f_const, nodal_f, gJ


def problems(i):
    dim, nx, ny, nz, batch, m, mode, flags, f_const, nodal_f, gJ = draw(i)
    inp = inputs.random_inputs(dim, nx, ny, nz, batch, m, seed=7000 + i, f_const=f_const)
    u = inputs.random_field(inp.u.shape, 50 + i)
    nu = inputs.random_positive_field(inp.u.shape, 60 + i) if mode == B.DN_NU_NODAL else None
    f = inputs.random_field(inp.u.shape, 70 + i, scale=2.0) if nodal_f else None
    po, pg = make_problems(inp, mode, nu=nu, f=f, flags=flags, bc=(0.6, -0.2))
    return po, pg, u, gJ


@pytest.mark.parametrize("i", range(N_CASES))
def test_random_problem(i):
    po, pg, u, gJ = problems(i)
    what = f"case {i}: {pg.shape} mode {pg.nu_mode} flags {pg.flags} path {B.dn_path_name(pg)}"
    Jo, _, _, ro = oracle.energy_grad(po, u, gJ=None if gJ is None else gJ.astype(np.float64))
    Jg, rg = run_gpu(pg, u, gJ=gJ)
    check(Jg, rg, Jo, ro, what)
    Jo1, _, _, _ = oracle.energy_grad(po, u)                     # the energy-only call takes no upstream gradient
    ws_n = max(B.dn_workspace_bytes(pg), 256)
    ws_whole, ws = guarded(ws_n)
    J = torch.empty(pg.batch, device="cuda")
    B.dn_energy(pg, dev(u), J, ws)
    torch.cuda.synchronize()
    assert guards_intact(ws_whole, ws_n), what
    rel = np.abs(J.cpu().numpy().astype(np.float64) - Jo1) / np.abs(Jo1)
    assert np.all(rel <= 1e-5), f"{what}: dn_energy rel err {rel.max():.2e}"


def test_the_seeds_reach_every_kernel_family():
    seen = set()
    for i in range(N_CASES):
        dim, nx, ny, nz, batch, m, mode, flags, f_const, nodal_f, gJ = draw(i)
        p = B.Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=batch, nu_mode=mode, kl_modes=m,
                      kl_w=torch.zeros((batch,) + (m,) * dim, device="cuda"),
                      nu=torch.ones(1, device="cuda") if mode == B.DN_NU_NODAL else None,
                      f=torch.ones(1, device="cuda") if nodal_f else None, flags=flags)
        seen.add(B.dn_path_name(p))
    assert seen == {"row2d", "strip2d", "tiled2d", "strip3d", "tiled3d", "generic"}
