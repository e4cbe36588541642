"""GPU parity: the CUDA library against the fp64 oracle, element by element, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, make_problems, run_gpu, check, J_RTOL, R_RTOL

pytestmark = pytest.mark.gpu

MODES = [B.DN_NU_KL_GAUSS, B.DN_NU_NODAL, B.DN_NU_KL_NODAL]


def nodal_nu(inp):
    """Nodal diffusivity for DN_NU_NODAL runs: the oracle's KL field rounded to float32."""
    return oracle.kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, inp.kl_w).astype(np.float32)


# ---- the workloads the oracle finishes in seconds, every node compared ---------------------------
@pytest.mark.parametrize("force_generic", [0, B.DN_FORCE_GENERIC])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("cfg", [0, 1, 3])
def test_workload_parity_full(cfg, mode, force_generic):
    inp = inputs.make_inputs(cfg)
    nu = nodal_nu(inp) if mode == B.DN_NU_NODAL else None
    po, pg = make_problems(inp, mode, nu=nu, flags=force_generic)
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    Jg, rg = run_gpu(pg, inp.u)
    check(Jg, rg, Jo, ro, f"cfg{cfg} mode{mode} path={B.dn_path_name(pg)}")
    assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)


# ---- odd sizes, ragged tails, degenerate extents --------------------------------------------------
ODD = [(2, 2, 2, 1, 1, 1), (2, 3, 2, 1, 2, 2), (2, 5, 9, 1, 3, 3), (2, 64, 7, 1, 2, 4), (2, 130, 67, 1, 2, 6),
       (2, 257, 33, 1, 1, 8), (2, 516, 40, 1, 2, 5), (2, 1028, 19, 1, 1, 2),
       (3, 2, 2, 2, 1, 1), (3, 3, 4, 5, 2, 2), (3, 9, 5, 7, 2, 3), (3, 36, 10, 6, 2, 2), (3, 132, 9, 5, 1, 3),
       (3, 64, 20, 3, 1, 2), (3, 260, 6, 4, 1, 2),
       # narrow 3D grids: a warp holds 4 rows (nx <= 32) or 2 rows (nx <= 64) of the tile; several tiles with seams
       (3, 12, 11, 6, 2, 2), (3, 32, 9, 7, 3, 3), (3, 28, 45, 5, 1, 2), (3, 60, 37, 6, 2, 3)]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dim,nx,ny,nz,batch,m", ODD)
def test_odd_sizes(dim, nx, ny, nz, batch, m, mode):
    inp = inputs.random_inputs(dim, nx, ny, nz, batch, m, seed=100 + nx + 7 * ny, f_const=0.6)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    for flags in (0, B.DN_FORCE_GENERIC):
        po, pg = make_problems(inp, mode, nu=nu, flags=flags)
        Jo, _, _, ro = oracle.energy_grad(po, inp.u)
        Jg, rg = run_gpu(pg, inp.u)
        check(Jg, rg, Jo, ro, f"{dim}d {nx}x{ny}x{nz} mode{mode} path={B.dn_path_name(pg)}")


# ---- options: on-load boundary values, no mask, upstream gradient, nodal forcing, energy only -----
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dim,nx,ny,nz", [(2, 128, 37, 1), (2, 50, 21, 1), (3, 64, 9, 6), (3, 17, 6, 5)])
def test_options(dim, nx, ny, nz, mode):
    inp = inputs.random_inputs(dim, nx, ny, nz, 3, 3, seed=42, f_const=-0.4)
    nu = inputs.random_positive_field(inp.u.shape, 6) if mode == B.DN_NU_NODAL else None
    u = inputs.random_field(inp.u.shape, 8)           # boundary values NOT satisfied
    gJ = np.array([1.5, -2.0, 0.25], dtype=np.float32)
    for flags in (0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK):
        for fg in (0, B.DN_FORCE_GENERIC):
            po, pg = make_problems(inp, mode, nu=nu, flags=flags | fg, bc=(0.8, -0.3))
            Jo, _, _, ro = oracle.energy_grad(po, u, gJ=gJ.astype(np.float64))
            Jg, rg = run_gpu(pg, u, gJ=gJ)
            check(Jg, rg, Jo, ro, f"flags={flags | fg}")
            if not (flags & B.DN_NO_MASK):
                assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)
    # nodal forcing (Q1-interpolated)
    f = inputs.random_field(inp.u.shape, 9)
    po, pg = make_problems(inp, mode, nu=nu, f=f)
    Jo, _, _, ro = oracle.energy_grad(po, u)
    Jg, rg = run_gpu(pg, u)
    check(Jg, rg, Jo, ro, "nodal f")
    # dn_energy == J of dn_energy_grad up to rounding; a residual-only call gives the same residual
    po, pg = make_problems(inp, mode, nu=nu)
    ws = B.new_workspace(pg)
    J1 = torch.empty(3, device="cuda"); J2 = torch.empty(3, device="cuda"); r = torch.empty(pg.shape, device="cuda")
    B.dn_energy(pg, dev(u), J1, ws)
    B.dn_energy_grad(pg, dev(u), None, J2, r, ws)
    r2 = torch.empty_like(r)
    B.dn_energy_grad(pg, dev(u), None, None, r2, ws)
    torch.cuda.synchronize()
    assert torch.allclose(J1, J2, rtol=1e-5, atol=0) and torch.equal(r, r2)


def test_apply_bc_then_grad_equals_impose_on_load():
    inp = inputs.random_inputs(2, 256, 40, 1, 2, 2, seed=3)
    u = inputs.random_field(inp.u.shape, 1)
    _, pg = make_problems(inp, B.DN_NU_KL_GAUSS, flags=B.DN_IMPOSE_BC_ON_LOAD, bc=(0.5, 0.25))
    Ja, ra = run_gpu(pg, u)
    ud = dev(u)
    B.dn_apply_bc(2, 256, 40, 1, 2, 0.5, 0.25, 0, ud)
    pg.flags = 0
    r = torch.empty(pg.shape, device="cuda"); J = torch.empty(2, device="cuda")
    B.dn_energy_grad(pg, ud, None, J, r, B.new_workspace(pg))
    torch.cuda.synchronize()
    assert np.array_equal(J.cpu().numpy(), Ja.astype(np.float32)) and np.array_equal(r.cpu().numpy(), ra.astype(np.float32))


@pytest.mark.parametrize("dim,nx,ny,nz,batch", [(2, 64, 9, 1, 3), (2, 7, 5, 1, 2), (3, 12, 5, 4, 2), (3, 5, 3, 2, 1)])
def test_apply_bc_bit_exact(dim, nx, ny, nz, batch):
    shape = (batch, nz, ny, nx) if dim == 3 else (batch, ny, nx)
    a = inputs.random_field(shape, 2)
    for mode in (0, 1):
        ref = oracle.apply_bc(dim, nx, ny, nz, batch, 0.7, -1.25, mode, a.copy())
        d = dev(a)
        B.dn_apply_bc(dim, nx, ny, nz, batch, 0.7, -1.25, mode, d)
        assert np.array_equal(d.cpu().numpy(), ref)


@pytest.mark.parametrize("dim,nx,ny,nz,batch,m", [(2, 64, 64, 1, 8, 2), (2, 256, 100, 1, 3, 6), (2, 37, 11, 1, 2, 8),
                                                  (3, 64, 20, 9, 2, 2), (3, 256, 17, 5, 1, 3), (3, 10, 7, 5, 2, 4)])
def test_kl_field_parity(dim, nx, ny, nz, batch, m):
    rng = np.random.default_rng(m + nx)
    w = np.stack([inputs.draw_weights(rng, dim, m) for _ in range(batch)])
    ref = oracle.kl_field(dim, nx, ny, nz, batch, m, w)
    out = torch.empty((batch, nz, ny, nx) if dim == 3 else (batch, ny, nx), device="cuda")
    B.dn_kl_field(dim, nx, ny, nz, batch, m, dev(w), out)
    got = out.cpu().numpy().astype(np.float64)
    assert np.abs(got / ref - 1).max() < 1e-5


def test_determinism_and_workspace_reuse():
    for cfg in (0, 3):
        inp = inputs.make_inputs(cfg)
        _, pg = make_problems(inp, B.DN_NU_KL_GAUSS)
        ws = B.new_workspace(pg)
        ud = dev(inp.u)
        outs = []
        for it in range(3):
            ws.fill_(255 if it == 1 else 0)                     # stale workspace contents must not matter
            r = torch.empty(pg.shape, device="cuda"); J = torch.empty(pg.batch, device="cuda")
            B.dn_energy_grad(pg, ud, None, J, r, ws)
            outs.append((J.cpu().numpy().copy(), r.cpu().numpy().copy()))
        for J, r in outs[1:]:
            assert J.tobytes() == outs[0][0].tobytes() and r.tobytes() == outs[0][1].tobytes()


def test_host_buffer_entry_point():
    inp = inputs.make_inputs(0)
    po, pg = make_problems(inp, B.DN_NU_KL_GAUSS)
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    ph = B.Problem(dim=2, nx=64, ny=64, batch=8, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2,
                   kl_w=torch.from_numpy(inp.kl_w).pin_memory(), bc_x0=1.0, bc_x1=0.0)
    u_h = torch.from_numpy(inp.u).pin_memory()
    r_h = torch.empty(pg.shape).pin_memory(); J_h = torch.empty(8).pin_memory()
    B.dn_energy_grad_host(ph, u_h, None, J_h, r_h, B.new_host_staging(ph))
    check(J_h.numpy().astype(np.float64), r_h.numpy().astype(np.float64), Jo, ro, "host entry")
    Jg, rg = run_gpu(pg, inp.u)
    assert np.array_equal(r_h.numpy(), rg.astype(np.float32))


def test_closed_form_on_gpu():
    """u = 1 - x, nu = c: J = c/2 and r = 0 away from the Dirichlet faces (no oracle involved)."""
    for dim, n in ((2, 256), (3, 64)):
        shape = (2,) + (n,) * dim
        u = np.broadcast_to((1 - np.arange(n) / (n - 1)).astype(np.float32), shape).copy()
        pg = B.Problem(dim=dim, nx=n, ny=n, nz=n if dim == 3 else 1, batch=2, nu_mode=B.DN_NU_NODAL,
                       nu=torch.full(shape, 2.5, device="cuda"))
        Jg, rg = run_gpu(pg, u)
        assert np.allclose(Jg, 1.25, rtol=1e-5)
        assert np.abs(rg).max() < 1e-5 * 2.5 / n


def test_side_stream_and_graph_replay():
    """Work is enqueued on the caller's stream only, and a captured dn_energy_grad replays to the same bits."""
    for cfg, samples in ((1, range(4)), (3, range(2))):
        inp = inputs.make_inputs(cfg, samples=samples)
        _, pg = make_problems(inp, B.DN_NU_KL_GAUSS)
        ud = dev(inp.u)
        ws = B.new_workspace(pg)
        r0 = torch.empty(pg.shape, device="cuda"); J0 = torch.empty(pg.batch, device="cuda")
        B.dn_energy_grad(pg, ud, None, J0, r0, ws)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        r1 = torch.zeros_like(r0); J1 = torch.zeros_like(J0)
        with torch.cuda.stream(side):
            B.dn_energy_grad(pg, ud, None, J1, r1, ws)
        side.synchronize()
        assert torch.equal(r0, r1) and torch.equal(J0, J1)
        r2 = torch.zeros_like(r0); J2 = torch.zeros_like(J0)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            B.dn_energy_grad(pg, ud, None, J2, r2, ws)
        r2.zero_(); J2.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(r0, r2) and torch.equal(J0, J2)
