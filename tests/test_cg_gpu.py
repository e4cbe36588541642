"""GPU parity of the matrix-free conjugate-gradient solver (dn_cg_solve) against the oracle's direct solve of the
assembled system K(nu) u = F with the Dirichlet faces eliminated."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs

pytestmark = pytest.mark.gpu

U_RTOL = 2e-4     # max |u - u*| <= U_RTOL max |u*| per sample (fp32 CG; the direct solve is fp64)
J_RTOL = 1e-5     # |J(u) - J(u*)| <= J_RTOL |J(u*)|

MODES = {"kl": (B.DN_NU_KL_GAUSS, oracle.NU_KL_GAUSS), "nodal": (B.DN_NU_NODAL, oracle.NU_NODAL),
         "klnodal": (B.DN_NU_KL_NODAL, oracle.NU_KL_NODAL)}


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def direct(inp, omode, nu, f, f_const, bc):
    us, Js = [], []
    for b in range(inp.batch):
        pb = oracle.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=1, nu_mode=omode,
                            nu=None if nu is None else nu[b:b + 1], kl_modes=inp.kl_modes, kl_w=inp.kl_w[b:b + 1],
                            f_const=f_const, f=None if f is None else f[b:b + 1], bc_x0=bc[0], bc_x1=bc[1])
        K, F = oracle.assemble(pb)
        u = oracle.solve_dirichlet(pb, K, F)
        us.append(u)
        Js.append(oracle.energy_grad(pb, u[None], want_r=False)[0][0])
    return np.stack(us), np.array(Js)


def solve(inp, mode, f=None, f_const=1.0, bc=(1.0, 0.0), iters=400, rtol=1e-6, flags=0, u0=None):
    gmode, omode = MODES[mode]
    nu = None
    if mode == "nodal":
        nu = oracle.kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, inp.kl_w).astype(np.float32)
    p = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=gmode, nu=dev(nu),
                  kl_modes=inp.kl_modes, kl_w=dev(inp.kl_w), f_const=f_const, f=dev(f), bc_x0=bc[0], bc_x1=bc[1], flags=flags)
    u = dev(inp.u if u0 is None else u0)
    relres = torch.full((inp.batch,), float("nan"), device="cuda")
    its = torch.full((inp.batch,), -1, dtype=torch.int32, device="cuda")
    B.dn_cg_solve(p, u, iters, rtol, relres, its, B.new_cg_workspace(p))
    torch.cuda.synchronize()
    return p, u, relres.cpu().numpy(), its.cpu().numpy(), (omode, nu)


CASES = [  # dim, nx, ny, nz, batch, mode, flags
    (2, 16, 16, 1, 3, "kl", 0), (2, 32, 24, 1, 2, "nodal", 0), (2, 21, 18, 1, 2, "kl", 0),
    (2, 24, 24, 1, 2, "klnodal", 0), (2, 16, 16, 1, 2, "kl", B.DN_FORCE_GENERIC),
    (3, 8, 8, 8, 2, "kl", 0), (3, 12, 8, 10, 2, "nodal", 0), (3, 9, 7, 6, 2, "kl", 0),
]


@pytest.mark.parametrize("dim,nx,ny,nz,batch,mode,flags", CASES)
def test_cg_reaches_the_direct_solution(dim, nx, ny, nz, batch, mode, flags):
    inp = inputs.random_inputs(dim, nx, ny, nz, batch, 2, seed=31 + nx + 7 * dim, f_const=1.0)
    p, u, relres, its, (omode, nu) = solve(inp, mode, f_const=1.5, bc=(0.75, -0.25), flags=flags)
    us, Js = direct(inp, omode, nu, None, 1.5, (0.75, -0.25))
    ug = u.cpu().numpy().astype(np.float64)
    assert np.all(relres <= 2e-6) and np.all(its > 0) and np.all(its < 400), (relres, its)
    for b in range(batch):
        assert np.abs(ug[b] - us[b]).max() <= U_RTOL * np.abs(us[b]).max(), np.abs(ug[b] - us[b]).max()
    assert np.all(ug[..., 0] == np.float32(0.75)) and np.all(ug[..., -1] == np.float32(-0.25))
    J = torch.empty(batch, device="cuda")
    r = torch.empty_like(u)
    B.dn_energy_grad(p, u, None, J, r, B.new_workspace(p))
    Jg = J.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(Jg - Js) <= J_RTOL * np.abs(Js)), (Jg, Js)
    assert np.all(Jg >= Js - J_RTOL * np.abs(Js))                       # nothing lies below the minimum


def test_cg_with_nodal_forcing_and_zero_iterations():
    inp = inputs.random_inputs(2, 20, 16, 1, 2, 2, seed=9, f_const=0.0)
    f = inputs.random_field((2, 16, 20), seed=10).astype(np.float32)
    p, u, relres, its, (omode, nu) = solve(inp, "kl", f=f, f_const=0.0)
    us, _ = direct(inp, omode, nu, f, 0.0, (1.0, 0.0))
    ug = u.cpu().numpy().astype(np.float64)
    assert np.abs(ug - us).max() <= U_RTOL * np.abs(us).max()
    p, u0, relres, its, _ = solve(inp, "kl", iters=0)
    ref = inp.u.copy(); ref[..., 0] = 1.0; ref[..., -1] = 0.0
    assert np.array_equal(u0.cpu().numpy(), ref) and np.all(its == 0) and np.all(relres == 1.0)


def _oracle_residual(inp, omode, nu, f, f_const, bc, u):
    po = oracle.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=omode, nu=nu,
                        kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=f_const, f=f, bc_x0=bc[0], bc_x1=bc[1])
    return oracle.energy_grad(po, u)


@pytest.mark.parametrize("nx,ny,mode,with_f", [(1024, 24, "kl", False), (2052, 17, "kl", False), (1024, 24, "klnodal", False),
                                                (1024, 24, "nodal", False), (1024, 24, "kl", True)])
def test_cg_on_wide_rows_where_the_strip_kernel_is_the_operator(nx, ny, mode, with_f):
    """Grids too large for a dense direct solve: the result is checked through the oracle's own residual and energy.
    CG started from a random field (|r0| = O(1) per node) must bring the oracle's residual of the returned field
    below 3e-5 |r0| -- it would not if the operator the iteration applies were not the oracle's K(nu) -- and the
    energy the library reports for that field must be the oracle's.  With nodal forcing the caller's problem runs on
    another kernel family than the direction operator, which still reads the tables built for it."""
    inp = inputs.random_inputs(2, nx, ny, 1, 2, 3, seed=50 + ny, sigma=1.0)
    f = inputs.random_field((2, ny, nx), seed=12).astype(np.float32) if with_f else None
    bc = (0.75, -0.25)
    p, u, relres, its, (omode, nu) = solve(inp, mode, f=f, f_const=1.5, bc=bc, iters=30000, rtol=1e-5)
    pd = B.Problem(dim=2, nx=nx, ny=ny, nz=1, batch=2, nu_mode=p.nu_mode, nu=p.nu, kl_modes=3, kl_w=p.kl_w)
    assert B.dn_path_name(pd) == "strip2d"
    assert np.all(relres <= 1e-5) and np.all(its < 30000), (relres, its)
    u0 = inp.u.copy(); u0[..., 0] = bc[0]; u0[..., -1] = bc[1]
    _, _, _, r0 = _oracle_residual(inp, omode, nu, f, 1.5, bc, u0)
    ug = u.cpu().numpy()
    Jo, _, _, ro = _oracle_residual(inp, omode, nu, f, 1.5, bc, ug)
    for b in range(2):
        assert np.linalg.norm(ro[b]) <= 3e-5 * np.linalg.norm(r0[b]), (np.linalg.norm(ro[b]), np.linalg.norm(r0[b]))
    assert np.all(ug[..., 0] == np.float32(bc[0])) and np.all(ug[..., -1] == np.float32(bc[1]))
    J = torch.empty(2, device="cuda"); r = torch.empty_like(u)
    B.dn_energy_grad(p, u, None, J, r, B.new_workspace(p))
    assert np.all(np.abs(J.cpu().numpy() - Jo) <= J_RTOL * np.abs(Jo))


def test_cg_is_deterministic_and_freezes_converged_samples():
    inp = inputs.random_inputs(2, 32, 32, 1, 3, 2, seed=3, f_const=1.0)
    _, ua, ra, ia, _ = solve(inp, "kl", iters=300, rtol=1e-4)
    _, ub, rb, ib, _ = solve(inp, "kl", iters=300, rtol=1e-4)
    assert torch.equal(ua, ub) and np.array_equal(ia, ib)
    _, uc, rc, ic, _ = solve(inp, "kl", iters=600, rtol=1e-4)                 # more iterations change nothing once frozen
    assert torch.equal(ua, uc) and np.array_equal(ia, ic) and np.all(ia < 300) and np.all(ra <= 1e-4)


def test_cg_validation():
    inp = inputs.random_inputs(2, 16, 16, 1, 1, 2, seed=3)
    p = B.Problem(dim=2, nx=16, ny=16, nz=1, batch=1, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=dev(inp.kl_w))
    u = dev(inp.u)
    with pytest.raises(B.DnError) as e:
        B.dn_cg_solve(p, u, 10, 1e-6, None, None, B.new_cg_workspace(p)[:256])
    assert e.value.status == B.DN_ERR_WORKSPACE
    with pytest.raises(B.DnError) as e:
        B.dn_cg_solve(p, u, -1, 1e-6, None, None, B.new_cg_workspace(p))
    assert e.value.status == B.DN_ERR_MODE
    assert B.dn_cg_workspace_bytes(B.Problem(dim=4, nx=16, ny=16, nz=1, batch=1, kl_modes=2, kl_w=dev(inp.kl_w))) == 0
