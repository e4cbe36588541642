"""GPU parity of the 3D strip kernel (rows of at most 256 nodes, energy and residual fused, all three diffusivity
modes) against the fp64 oracle: every lane layout (4 or 8 nodes per lane; 8, 16 or 32 lanes per unit, i.e. 4, 2 or 1
units per warp), rows that end inside a lane group, one and many tiles and chunks, batches that leave units of a warp
idle, and every option the kernel serves."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, make_problems, run_gpu, check, guarded, guards_intact

pytestmark = pytest.mark.gpu

# (nx, ny, nz, batch, m)
SIZES = [(8, 2, 2, 1, 1), (12, 11, 6, 2, 2), (32, 9, 7, 3, 3), (28, 45, 5, 1, 2), (36, 10, 6, 5, 2), (64, 20, 3, 1, 2),
         (60, 37, 6, 2, 3), (64, 64, 17, 3, 2), (100, 7, 9, 2, 4), (128, 13, 12, 1, 8), (132, 9, 5, 1, 3), (136, 6, 7, 2, 2),
         (200, 5, 4, 1, 5), (256, 17, 5, 1, 3), (256, 40, 30, 2, 6), (64, 150, 40, 9, 2), (16, 8, 300, 1, 1),
         # rows of 65 to 128 nodes that are a multiple of 8: 8 nodes per lane and two units per warp (KL at the Gauss points)
         (72, 9, 7, 3, 2), (96, 20, 5, 2, 3), (120, 6, 6, 1, 4), (128, 40, 9, 5, 2), (88, 3, 30, 7, 1)]


MODES = [B.DN_NU_KL_GAUSS, B.DN_NU_KL_NODAL, B.DN_NU_NODAL]   # KL at the Gauss points / at the nodes (in the kernel), stored nodal field


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("nx,ny,nz,batch,m", SIZES)
def test_strip3d_parity(nx, ny, nz, batch, m, mode):
    inp = inputs.random_inputs(3, nx, ny, nz, batch, m, seed=11 + nx + 3 * ny + nz, f_const=0.6)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    po, pg = make_problems(inp, mode, nu=nu)
    expect = "strip3d" if (nx <= 128 or nx % 8 == 0) else ("generic" if mode == B.DN_NU_KL_NODAL else "tiled3d")
    assert B.dn_path_name(pg) == expect
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    Jg, rg = run_gpu(pg, inp.u)
    check(Jg, rg, Jo, ro, f"strip3d {nx}x{ny}x{nz} b{batch} m{m}")
    assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("nx,ny,nz", [(64, 9, 6), (24, 6, 5), (256, 7, 6), (128, 12, 9)])
def test_strip3d_options(nx, ny, nz, mode):
    inp = inputs.random_inputs(3, nx, ny, nz, 3, 3, seed=42, f_const=-0.4)
    u = inputs.random_field(inp.u.shape, 8)           # boundary values NOT satisfied
    nu = inputs.random_positive_field(inp.u.shape, 6) if mode == B.DN_NU_NODAL else None
    gJ = np.array([1.5, -2.0, 0.25], dtype=np.float32)
    for flags in (0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK):
        po, pg = make_problems(inp, mode, nu=nu, flags=flags, bc=(0.8, -0.3))
        assert B.dn_path_name(pg) == "strip3d"
        Jo, _, _, ro = oracle.energy_grad(po, u, gJ=gJ.astype(np.float64))
        Jg, rg = run_gpu(pg, u, gJ=gJ)
        check(Jg, rg, Jo, ro, f"flags={flags}")
        if not (flags & B.DN_NO_MASK):
            assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)
    # rectangular cells (hx != hy != hz take the scaled path), residual-only call, determinism with a stale workspace
    po, pg = make_problems(inp, mode, nu=nu)
    ws = B.new_workspace(pg)
    outs = []
    for it in range(3):
        ws.fill_(255 if it == 1 else 0)
        r = torch.empty(pg.shape, device="cuda"); J = torch.empty(3, device="cuda")
        B.dn_energy_grad(pg, dev(u), None, J if it < 2 else None, r, ws)
        torch.cuda.synchronize()
        outs.append((J.cpu().numpy().copy(), r.cpu().numpy().copy()))
    assert outs[0][0].tobytes() == outs[1][0].tobytes()
    assert outs[0][1].tobytes() == outs[1][1].tobytes() == outs[2][1].tobytes()
    J1 = torch.empty(3, device="cuda")
    B.dn_energy(pg, dev(u), J1, ws)                   # the energy-only call runs another kernel family
    assert np.allclose(J1.cpu().numpy(), outs[0][0], rtol=1e-5, atol=0)


def test_strip3d_isotropic_cells_and_closed_form():
    """Cubic cells take the unscaled path; u = 1 - x with all weights zero (nu = 1) has J = 1/2 and r = 0 off the faces."""
    n = 48
    u = np.broadcast_to((1 - np.arange(n) / (n - 1)).astype(np.float32), (2, n, n, n)).copy()
    pg = B.Problem(dim=3, nx=n, ny=n, nz=n, batch=2, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2,
                   kl_w=torch.zeros(2, 2, 2, 2, device="cuda"))
    assert B.dn_path_name(pg) == "strip3d"
    Jg, rg = run_gpu(pg, u)
    assert np.allclose(Jg, 0.5, rtol=1e-5)
    assert np.abs(rg).max() < 1e-5 / n


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("nx,ny,nz,batch,m", [(64, 20, 9, 3, 2), (24, 7, 6, 2, 3), (256, 12, 7, 1, 3), (128, 9, 13, 2, 4), (136, 6, 5, 1, 2)])
def test_strip3d_nodal_forcing(nx, ny, nz, batch, m, mode):
    """Nodal forcing on the 3D strip kernel: the load is taken element by element (mass matrix applied to the corner values
    of f) and gathered with the stiffness contributions, across tile and chunk seams; anisotropic cells; every flag."""
    inp = inputs.random_inputs(3, nx, ny, nz, batch, m, seed=23 + nx + ny)
    u = inputs.random_field(inp.u.shape, 4)
    f = inputs.random_field(inp.u.shape, 9, scale=3.0)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    gJ = np.linspace(-1.5, 2.0, batch).astype(np.float32)
    for flags in (0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD):
        po, pg = make_problems(inp, mode, nu=nu, f=f, flags=flags, bc=(0.8, -0.3))
        assert B.dn_path_name(pg) == "strip3d"
        Jo, _, _, ro = oracle.energy_grad(po, u, gJ=gJ.astype(np.float64))
        Jg, rg = run_gpu(pg, u, gJ=gJ)
        check(Jg, rg, Jo, ro, f"nodal f, flags={flags}")
        if not (flags & B.DN_NO_MASK):
            assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)


def test_strip3d_nodal_forcing_on_cubic_cells():
    inp = inputs.random_inputs(3, 40, 40, 40, 2, 2, seed=5)
    f = inputs.random_field(inp.u.shape, 3)
    po, pg = make_problems(inp, B.DN_NU_KL_GAUSS, f=f)
    assert B.dn_path_name(pg) == "strip3d"
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    Jg, rg = run_gpu(pg, inp.u)
    check(Jg, rg, Jo, ro, "nodal f, cubic cells")


@pytest.mark.parametrize("seed", range(36))
def test_strip3d_random_shapes(seed):
    """Seeded random shapes, modes, flags and forcing kinds: tiles and chunks with ragged ends, single-row tiles, one-plane
    chunks, every lane layout, m up to 8 (the coefficient row then needs more pieces than a narrow unit has lanes)."""
    rng = np.random.default_rng(1000 + seed)
    nx = int(rng.choice([8, 12, 16, 24, 32, 36, 48, 64, 72, 100, 128, 136, 192, 256]))
    ny, nz = int(rng.integers(2, 34)), int(rng.integers(2, 34))
    if nx >= 128:
        ny, nz = min(ny, 14), min(nz, 14)
    batch, m = int(rng.integers(1, 6)), int(rng.integers(1, 9))
    mode = MODES[int(rng.integers(0, 3))]
    flags = int(rng.choice([0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK]))
    inp = inputs.random_inputs(3, nx, ny, nz, batch, m, seed=2000 + seed, f_const=float(rng.choice([0.0, 0.7])))
    u = inputs.random_field(inp.u.shape, 50 + seed)
    nu = inputs.random_positive_field(inp.u.shape, 60 + seed) if mode == B.DN_NU_NODAL else None
    f = inputs.random_field(inp.u.shape, 70 + seed, scale=2.0) if rng.random() < 0.4 else None
    gJ = rng.uniform(-2, 2, batch).astype(np.float32) if rng.random() < 0.5 else None
    po, pg = make_problems(inp, mode, nu=nu, f=f, flags=flags, bc=(0.6, -0.2))
    assert B.dn_path_name(pg) == "strip3d"
    Jo, _, _, ro = oracle.energy_grad(po, u, gJ=None if gJ is None else gJ.astype(np.float64))
    Jg, rg = run_gpu(pg, u, gJ=gJ)
    check(Jg, rg, Jo, ro, f"seed {seed}: {nx}x{ny}x{nz} b{batch} m{m} mode{mode} flags{flags} f={'nodal' if f is not None else inp.f_const}")


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("nx,ny,nz,batch,m", [(8, 2, 2, 1, 1), (12, 11, 6, 2, 2), (36, 10, 6, 5, 2), (64, 64, 17, 3, 2), (128, 13, 12, 1, 8),
                                              (136, 6, 7, 2, 2), (256, 17, 5, 1, 3), (256, 40, 30, 2, 6), (16, 8, 300, 1, 1)])
def test_strip3d_energy_only(nx, ny, nz, batch, m, mode):
    """dn_energy runs the same march without the gather (every element adds its own energy): against the oracle's J, with
    constant and with nodal forcing, cubic and stretched cells, boundary values imposed on load."""
    inp = inputs.random_inputs(3, nx, ny, nz, batch, m, seed=31 + nx + ny + nz, f_const=0.6)
    u = inputs.random_field(inp.u.shape, 12)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    f = inputs.random_field(inp.u.shape, 9, scale=3.0)
    for ff, flags in ((None, 0), (None, B.DN_IMPOSE_BC_ON_LOAD), (f, 0), (f, B.DN_IMPOSE_BC_ON_LOAD)):
        po, pg = make_problems(inp, mode, nu=nu, f=ff, flags=flags, bc=(0.8, -0.3))
        assert B.dn_path_name(pg) == "strip3d"
        Jo, _, _, _ = oracle.energy_grad(po, u)
        ws_n = max(B.dn_workspace_bytes(pg), 256)
        ws_whole, ws = guarded(ws_n)
        J_whole, J_bytes = guarded(4 * batch)
        J = J_bytes.view(torch.float32)
        B.dn_energy(pg, dev(u), J, ws)
        torch.cuda.synchronize()
        assert guards_intact(ws_whole, ws_n) and guards_intact(J_whole, 4 * batch)
        rel = np.abs(J.cpu().numpy().astype(np.float64) - Jo) / np.abs(Jo)
        assert np.all(rel <= 1e-5), f"{nx}x{ny}x{nz} mode {mode} f={'nodal' if ff is not None else 'const'} flags={flags}: {rel.max():.2e}"


def test_strip3d_energy_only_on_cubic_cells_matches_the_fused_call():
    inp = inputs.random_inputs(3, 48, 48, 48, 3, 2, seed=77, f_const=1.0)
    for mode in MODES:
        nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
        po, pg = make_problems(inp, mode, nu=nu)
        Jo, _, _, _ = oracle.energy_grad(po, inp.u)
        Jg, _ = run_gpu(pg, inp.u)
        J = torch.empty(3, device="cuda")
        B.dn_energy(pg, dev(inp.u), J, B.new_workspace(pg))
        Je = J.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(Je - Jo) <= 1e-5 * np.abs(Jo)) and np.all(np.abs(Je - Jg) <= 2e-6 * np.abs(Jo))
