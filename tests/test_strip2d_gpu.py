"""GPU parity of the strip kernel (2D, KL diffusivity at the Gauss points, energy and residual fused) against the
fp64 oracle: strips that end exactly at the grid, ragged last strips, one and many chunks, every option it serves."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, make_problems, run_gpu, check, guarded, guards_intact

pytestmark = pytest.mark.gpu

# (nx, ny, batch, m): the kernel takes rows from about 1000 nodes on (narrower ones waste too many lanes) and every
# width beyond the tiled kernel's 2048.  124 k + 128 = 1120 ends a strip exactly at the grid; 1116 / 1124 are one lane
# short / one lane beyond; 2048 is the bench width; 2052 and 4096 only this kernel and the any-size kernels can run;
# ny = 16 is the shortest grid, 700 rows span several chunks
SIZES = [(1024, 40, 2, 4), (1028, 17, 3, 1), (1116, 33, 2, 6), (1120, 16, 2, 2), (1124, 21, 1, 3), (1500, 50, 2, 5),
         (2048, 24, 2, 8), (2052, 37, 1, 7), (4096, 19, 2, 6), (1024, 700, 10, 2)]


KL_MODES = [B.DN_NU_KL_GAUSS, B.DN_NU_KL_NODAL, B.DN_NU_NODAL]   # KL at the Gauss points / at the nodes (in the kernel), stored nodal field


@pytest.mark.parametrize("mode", KL_MODES)
@pytest.mark.parametrize("nx,ny,batch,m", SIZES)
def test_strip2d_parity(nx, ny, batch, m, mode):
    inp = inputs.random_inputs(2, nx, ny, 1, batch, m, seed=7 + nx + ny, f_const=0.6)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    po, pg = make_problems(inp, mode, nu=nu)
    assert B.dn_path_name(pg) == "strip2d"
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    Jg, rg = run_gpu(pg, inp.u)
    check(Jg, rg, Jo, ro, f"strip2d {nx}x{ny} b{batch} m{m}")
    assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)
    # the any-size kernels on the same problem: two independent CUDA paths agree with the oracle
    _, pgen = make_problems(inp, mode, nu=nu, flags=B.DN_FORCE_GENERIC)
    Jg2, rg2 = run_gpu(pgen, inp.u)
    check(Jg2, rg2, Jo, ro, "generic")


@pytest.mark.parametrize("mode", KL_MODES)
@pytest.mark.parametrize("nx,ny", [(1024, 37), (1120, 19), (2500, 23)])
def test_strip2d_options(nx, ny, mode):
    inp = inputs.random_inputs(2, nx, ny, 1, 3, 3, seed=42, f_const=-0.4)
    u = inputs.random_field(inp.u.shape, 8)           # boundary values NOT satisfied
    nu = inputs.random_positive_field(inp.u.shape, 6) if mode == B.DN_NU_NODAL else None
    gJ = np.array([1.5, -2.0, 0.25], dtype=np.float32)
    for flags in (0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK):
        po, pg = make_problems(inp, mode, nu=nu, flags=flags, bc=(0.8, -0.3))
        assert B.dn_path_name(pg) == "strip2d"
        Jo, _, _, ro = oracle.energy_grad(po, u, gJ=gJ.astype(np.float64))
        Jg, rg = run_gpu(pg, u, gJ=gJ)
        check(Jg, rg, Jo, ro, f"flags={flags}")
        if not (flags & B.DN_NO_MASK):
            assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)
    # energy-only call (tiled kernel) against the fused call (strip kernel); residual-only call gives the same residual
    po, pg = make_problems(inp, mode, nu=nu)
    ws = B.new_workspace(pg)
    J1 = torch.empty(3, device="cuda"); J2 = torch.empty(3, device="cuda"); r = torch.empty(pg.shape, device="cuda")
    B.dn_energy(pg, dev(u), J1, ws)
    B.dn_energy_grad(pg, dev(u), None, J2, r, ws)
    r2 = torch.empty_like(r)
    B.dn_energy_grad(pg, dev(u), None, None, r2, ws)
    torch.cuda.synchronize()
    assert torch.allclose(J1, J2, rtol=1e-5, atol=0) and torch.equal(r, r2)


def test_strip2d_per_sample_boundary_values():
    inp = inputs.random_inputs(2, 1100, 18, 1, 3, 2, seed=5, f_const=0.3)
    u = inputs.random_field(inp.u.shape, 3)
    b0 = np.array([0.9, -0.2, 0.4], dtype=np.float32); b1 = np.array([0.1, 0.7, -0.6], dtype=np.float32)
    _, pg = make_problems(inp, B.DN_NU_KL_GAUSS, flags=B.DN_IMPOSE_BC_ON_LOAD)
    pg.bc_x0_b = dev(b0); pg.bc_x1_b = dev(b1)
    Jg, rg = run_gpu(pg, u)
    for s in range(3):                                 # the oracle, sample by sample with that sample's values
        one = inputs.random_inputs(2, 1100, 18, 1, 3, 2, seed=5, f_const=0.3)
        po = oracle.Problem(dim=2, nx=1100, ny=18, nz=1, batch=1, nu_mode=B.DN_NU_KL_GAUSS, nu=None, kl_modes=2,
                            kl_w=one.kl_w[s:s + 1], f_const=0.3, f=None, bc_x0=float(b0[s]), bc_x1=float(b1[s]),
                            flags=B.DN_IMPOSE_BC_ON_LOAD)
        Jo, _, _, ro = oracle.energy_grad(po, u[s:s + 1])
        check(Jg[s:s + 1], rg[s:s + 1], Jo, ro, f"sample {s}")


def test_strip2d_determinism_and_stale_workspace():
    inp = inputs.random_inputs(2, 1028, 300, 1, 2, 6, seed=11)
    _, pg = make_problems(inp, B.DN_NU_KL_GAUSS)
    ws = B.new_workspace(pg)
    ud = dev(inp.u)
    outs = []
    for it in range(3):
        ws.fill_(255 if it == 1 else 0)
        r = torch.empty(pg.shape, device="cuda"); J = torch.empty(pg.batch, device="cuda")
        B.dn_energy_grad(pg, ud, None, J, r, ws)
        outs.append((J.cpu().numpy().copy(), r.cpu().numpy().copy()))
    for J, r in outs[1:]:
        assert J.tobytes() == outs[0][0].tobytes() and r.tobytes() == outs[0][1].tobytes()


@pytest.mark.parametrize("mode", KL_MODES)
@pytest.mark.parametrize("nx,ny,batch,m", [(1024, 40, 2, 4), (1120, 16, 2, 2), (1124, 21, 1, 3), (2052, 37, 1, 7), (1024, 300, 5, 2),
                                           (256, 64, 3, 4), (380, 33, 2, 2),      # with nodal forcing also narrow rows
                                           (8, 16, 2, 1), (12, 40, 3, 2), (64, 64, 5, 3), (100, 17, 2, 4), (128, 33, 1, 8), (132, 20, 2, 2),
                                           (252, 50, 2, 5)])
def test_strip2d_nodal_forcing(nx, ny, batch, m, mode):
    """Nodal forcing on the strip kernel: the load vector is the consistent mass matrix applied to f (the f row rides in the
    ring with the u row).  All flag combinations, because the Dirichlet columns take the one-sided mass weights."""
    inp = inputs.random_inputs(2, nx, ny, 1, batch, m, seed=17 + nx + ny)
    u = inputs.random_field(inp.u.shape, 4)
    f = inputs.random_field(inp.u.shape, 9, scale=3.0)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    gJ = np.linspace(-1.5, 2.0, batch).astype(np.float32)
    for flags in (0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD):
        po, pg = make_problems(inp, mode, nu=nu, f=f, flags=flags, bc=(0.8, -0.3))
        assert B.dn_path_name(pg) == "strip2d"
        Jo, _, _, ro = oracle.energy_grad(po, u, gJ=gJ.astype(np.float64))
        Jg, rg = run_gpu(pg, u, gJ=gJ)
        check(Jg, rg, Jo, ro, f"nodal f, flags={flags}")
        if not (flags & B.DN_NO_MASK):
            assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)


@pytest.mark.parametrize("seed", range(24))
def test_strip2d_random_shapes(seed):
    """Seeded random shapes, modes, flags and forcing kinds on the 2D strip kernel."""
    rng = np.random.default_rng(3000 + seed)
    f_nodal = rng.random() < 0.5
    nx = 4 * int(rng.integers(2 if f_nodal else 250, 700))        # without nodal forcing rows below about 1000 nodes run tiled2d
    ny = int(rng.integers(16, 90))
    batch, m = int(rng.integers(1, 4)), int(rng.integers(1, 9))
    mode = KL_MODES[int(rng.integers(0, 3))]
    flags = int(rng.choice([0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK]))
    inp = inputs.random_inputs(2, nx, ny, 1, batch, m, seed=4000 + seed, f_const=float(rng.choice([0.0, 0.7])))
    u = inputs.random_field(inp.u.shape, 50 + seed)
    nu = inputs.random_positive_field(inp.u.shape, 60 + seed) if mode == B.DN_NU_NODAL else None
    f = inputs.random_field(inp.u.shape, 70 + seed, scale=2.0) if f_nodal else None
    gJ = rng.uniform(-2, 2, batch).astype(np.float32) if rng.random() < 0.5 else None
    po, pg = make_problems(inp, mode, nu=nu, f=f, flags=flags, bc=(0.6, -0.2))
    if B.dn_path_name(pg) != "strip2d":
        pytest.skip("this width takes the tiled kernel")
    Jo, _, _, ro = oracle.energy_grad(po, u, gJ=None if gJ is None else gJ.astype(np.float64))
    Jg, rg = run_gpu(pg, u, gJ=gJ)
    check(Jg, rg, Jo, ro, f"seed {seed}: {nx}x{ny} b{batch} m{m} mode{mode} flags{flags} f={'nodal' if f_nodal else inp.f_const}")


@pytest.mark.parametrize("mode", KL_MODES)
@pytest.mark.parametrize("nx,ny,batch,m", [(1024, 40, 2, 4), (1116, 33, 2, 6), (1120, 16, 2, 2), (1124, 21, 1, 3), (2052, 37, 1, 7),
                                           (4096, 19, 2, 6), (1024, 300, 5, 2), (256, 64, 3, 4)])
def test_strip2d_energy_only(nx, ny, batch, m, mode):
    """dn_energy on wide rows runs the same march without the gather (every element adds its own energy): against the
    oracle's J, with constant and with nodal forcing, boundary values imposed on load.  Rows of 256 nodes take this
    kernel with nodal forcing only."""
    inp = inputs.random_inputs(2, nx, ny, 1, batch, m, seed=19 + nx + ny, f_const=0.6)
    u = inputs.random_field(inp.u.shape, 12)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    f = inputs.random_field(inp.u.shape, 9, scale=3.0)
    for ff, flags in ((None, 0), (None, B.DN_IMPOSE_BC_ON_LOAD), (f, 0), (f, B.DN_IMPOSE_BC_ON_LOAD)):
        po, pg = make_problems(inp, mode, nu=nu, f=ff, flags=flags, bc=(0.8, -0.3))
        Jo, _, _, _ = oracle.energy_grad(po, u)
        ws_n = max(B.dn_workspace_bytes(pg), 256)
        ws_whole, ws = guarded(ws_n)
        J_whole, J_bytes = guarded(4 * batch)
        J = J_bytes.view(torch.float32)
        B.dn_energy(pg, dev(u), J, ws)
        torch.cuda.synchronize()
        assert guards_intact(ws_whole, ws_n) and guards_intact(J_whole, 4 * batch)
        rel = np.abs(J.cpu().numpy().astype(np.float64) - Jo) / np.abs(Jo)
        assert np.all(rel <= 1e-5), f"{nx}x{ny} mode {mode} f={'nodal' if ff is not None else 'const'} flags={flags}: {rel.max():.2e}"
