"""GPU parity of the 2D row kernel (rows of at most 256 nodes: a whole row per unit, energy and residual fused, all three
diffusivity modes, constant forcing) against the fp64 oracle: every lane layout (4 or 8 nodes per lane; 8, 16 or 32
lanes per unit, i.e. 4, 2 or 1 units per warp), rows that end inside a lane group, one and many chunks, batches that
leave units of a warp idle, and every option the kernel serves."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from parity_util import dev, make_problems, run_gpu, check

pytestmark = pytest.mark.gpu

# (nx, ny, batch, m)
SIZES = [(8, 2, 1, 1), (12, 11, 2, 2), (32, 9, 3, 3), (28, 45, 1, 2), (36, 10, 5, 2), (64, 64, 16, 4), (60, 37, 2, 3),
         (100, 7, 2, 4), (128, 13, 1, 8), (128, 300, 7, 2), (132, 9, 1, 3), (136, 6, 2, 2), (200, 5, 1, 5), (256, 17, 1, 3),
         (256, 256, 9, 4), (64, 1500, 3, 2), (16, 8, 70, 1), (256, 2, 1, 6)]

MODES = [B.DN_NU_KL_GAUSS, B.DN_NU_KL_NODAL, B.DN_NU_NODAL]   # KL at the Gauss points / at the nodes (in the kernel), stored nodal field


def expected_path(nx, mode):
    """Rows above 128 nodes take 8 nodes per lane: the KL modes only, and only rows that are a multiple of 8."""
    return "row2d" if (nx <= 128 or (nx % 8 == 0 and mode != B.DN_NU_NODAL)) else "tiled2d"


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("nx,ny,batch,m", SIZES)
def test_row2d_parity(nx, ny, batch, m, mode):
    inp = inputs.random_inputs(2, nx, ny, 1, batch, m, seed=11 + nx + 3 * ny, f_const=0.6)
    nu = inputs.random_positive_field(inp.u.shape, 5) if mode == B.DN_NU_NODAL else None
    po, pg = make_problems(inp, mode, nu=nu)
    assert B.dn_path_name(pg) == expected_path(nx, mode)
    Jo, _, _, ro = oracle.energy_grad(po, inp.u)
    Jg, rg = run_gpu(pg, inp.u)
    check(Jg, rg, Jo, ro, f"row2d {nx}x{ny} b{batch} m{m}")
    assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("nx,ny", [(64, 9), (24, 60), (256, 7), (128, 33)])
def test_row2d_options(nx, ny, mode):
    inp = inputs.random_inputs(2, nx, ny, 1, 3, 3, seed=42, f_const=-0.4)
    u = inputs.random_field(inp.u.shape, 8)           # boundary values NOT satisfied
    nu = inputs.random_positive_field(inp.u.shape, 6) if mode == B.DN_NU_NODAL else None
    gJ = np.array([1.5, -2.0, 0.25], dtype=np.float32)
    bc_b = (np.array([0.1, 0.5, -0.7], dtype=np.float32), np.array([0.9, -0.2, 0.3], dtype=np.float32))
    for flags in (0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK):
        po, pg = make_problems(inp, mode, nu=nu, flags=flags, bc=(0.8, -0.3))
        assert B.dn_path_name(pg) == expected_path(nx, mode)
        Jo, _, _, ro = oracle.energy_grad(po, u, gJ=gJ.astype(np.float64))
        Jg, rg = run_gpu(pg, u, gJ=gJ)
        check(Jg, rg, Jo, ro, f"flags={flags}")
        if not (flags & B.DN_NO_MASK):
            assert np.all(rg[..., 0] == 0.0) and np.all(rg[..., -1] == 0.0)
    # per-sample boundary values imposed on load
    _, pg = make_problems(inp, mode, nu=nu, flags=B.DN_IMPOSE_BC_ON_LOAD, bc=(0.8, -0.3))
    pg.bc_x0_b = dev(bc_b[0]); pg.bc_x1_b = dev(bc_b[1])
    Jg, rg = run_gpu(pg, u)
    for s in range(3):                                # the oracle takes one pair of values per call
        po = oracle.Problem(dim=2, nx=nx, ny=ny, nz=1, batch=1, nu_mode=mode, nu=None if nu is None else nu[s:s + 1],
                            kl_modes=3, kl_w=inp.kl_w[s:s + 1], f_const=-0.4, f=None, bc_x0=float(bc_b[0][s]),
                            bc_x1=float(bc_b[1][s]), flags=B.DN_IMPOSE_BC_ON_LOAD)
        Jo, _, _, ro = oracle.energy_grad(po, u[s:s + 1])
        check(Jg[s:s + 1], rg[s:s + 1], Jo, ro, f"per-sample boundary values, sample {s}")
    # residual-only call, determinism with a stale workspace
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


def test_row2d_closed_form():
    """u = 1 - x with all weights zero (nu = 1) has J = 1/2 and r = 0 off the Dirichlet columns."""
    n = 192
    u = np.broadcast_to((1 - np.arange(n) / (n - 1)).astype(np.float32), (2, n, n)).copy()
    pg = B.Problem(dim=2, nx=n, ny=n, batch=2, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=torch.zeros(2, 2, 2, device="cuda"))
    assert B.dn_path_name(pg) == "row2d"
    Jg, rg = run_gpu(pg, u)
    assert np.allclose(Jg, 0.5, rtol=1e-5)
    assert np.abs(rg).max() < 5e-7          # differences of the float values of u carry their rounding (an ulp of 1)


def test_row2d_and_the_any_size_kernel_agree_on_an_unaligned_view():
    """A field that starts 4 bytes off a 16-byte boundary cannot take the vector loads: the call falls back to the any-size
    kernel and must give the same numbers to rounding."""
    inp = inputs.random_inputs(2, 64, 40, 1, 2, 3, seed=9, f_const=0.3)
    po, pg = make_problems(inp, B.DN_NU_KL_GAUSS)
    Jg, rg = run_gpu(pg, inp.u)
    flat = torch.empty(inp.u.size + 1, device="cuda")
    uo = flat[1:].view(inp.u.shape)
    uo.copy_(dev(inp.u))
    r = torch.empty(pg.shape, device="cuda"); J = torch.empty(2, device="cuda")
    B.dn_energy_grad(pg, uo, None, J, r, B.new_workspace(pg))
    torch.cuda.synchronize()
    assert np.allclose(J.cpu().numpy(), Jg, rtol=1e-5)
    assert np.allclose(r.cpu().numpy(), rg, rtol=0, atol=1e-5 * np.abs(rg).max())


@pytest.mark.parametrize("seed", range(36))
def test_row2d_random_shapes(seed):
    """Seeded random shapes, modes and flags: chunks with ragged ends, two-row grids, every lane layout, m up to 8 (the
    coefficient row then needs more pieces than a narrow unit has lanes)."""
    rng = np.random.default_rng(5000 + seed)
    nx = int(rng.choice([8, 12, 16, 24, 32, 36, 48, 64, 72, 100, 128, 136, 192, 256]))
    ny = int(rng.integers(2, 400))
    batch, m = int(rng.integers(1, 40)), int(rng.integers(1, 9))
    mode = MODES[int(rng.integers(0, 3))]
    flags = int(rng.choice([0, B.DN_NO_MASK, B.DN_IMPOSE_BC_ON_LOAD, B.DN_IMPOSE_BC_ON_LOAD | B.DN_NO_MASK]))
    inp = inputs.random_inputs(2, nx, ny, 1, batch, m, seed=6000 + seed, f_const=float(rng.choice([0.0, 0.7])))
    u = inputs.random_field(inp.u.shape, 50 + seed)
    nu = inputs.random_positive_field(inp.u.shape, 60 + seed) if mode == B.DN_NU_NODAL else None
    gJ = rng.uniform(-2, 2, batch).astype(np.float32) if rng.random() < 0.5 else None
    po, pg = make_problems(inp, mode, nu=nu, flags=flags, bc=(0.6, -0.2))
    assert B.dn_path_name(pg) == expected_path(nx, mode)
    Jo, _, _, ro = oracle.energy_grad(po, u, gJ=None if gJ is None else gJ.astype(np.float64))
    Jg, rg = run_gpu(pg, u, gJ=gJ)
    check(Jg, rg, Jo, ro, f"seed {seed}: {nx}x{ny} b{batch} m{m} mode{mode} flags{flags} f={inp.f_const}")
