"""Per-sample Dirichlet values (the paper samples the boundary data b per minibatch): every kernel family reads
them when the faces are imposed on load, dn_apply_bc_per_sample writes them, dn_cg_solve solves with them.  The
oracle takes one pair of values per call, so it is called sample by sample."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs

pytestmark = pytest.mark.gpu


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


CASES = [(2, 64, 40, 1, 0), (2, 37, 21, 1, 0), (2, 64, 40, 1, B.DN_FORCE_GENERIC), (3, 16, 12, 10, 0), (3, 9, 7, 6, 0)]


@pytest.mark.parametrize("dim,nx,ny,nz,flags", CASES)
@pytest.mark.parametrize("which", ["both", "left_only"])
def test_faces_imposed_on_load_per_sample(dim, nx, ny, nz, flags, which):
    bs = 3
    inp = inputs.random_inputs(dim, nx, ny, nz, bs, 2, seed=41 + nx, f_const=0.5)
    b0 = np.array([1.0, -0.5, 2.25], dtype=np.float32)
    b1 = np.array([0.0, 0.75, -1.5], dtype=np.float32)
    p = B.Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=bs, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=dev(inp.kl_w),
                  f_const=0.5, bc_x0=9.0, bc_x1=0.3, flags=flags | B.DN_IMPOSE_BC_ON_LOAD,
                  bc_x0_b=dev(b0), bc_x1_b=dev(b1) if which == "both" else None)
    u = dev(inp.u)
    J = torch.empty(bs, device="cuda"); r = torch.empty_like(u)
    B.dn_energy_grad(p, u, None, J, r, B.new_workspace(p))
    torch.cuda.synchronize()
    for b in range(bs):
        po = oracle.Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=oracle.NU_KL_GAUSS, kl_modes=2,
                            kl_w=inp.kl_w[b:b + 1], f_const=0.5, bc_x0=float(b0[b]),
                            bc_x1=float(b1[b]) if which == "both" else float(np.float32(0.3)), flags=oracle.IMPOSE_BC_ON_LOAD)
        Jo, _, _, ro = oracle.energy_grad(po, inp.u[b:b + 1])
        assert abs(float(J[b]) - Jo[0]) <= 1e-5 * abs(Jo[0])
        assert np.abs(r[b].cpu().numpy() - ro[0]).max() <= 1e-5 * np.abs(ro).max()


def test_apply_bc_per_sample_and_validation():
    f = torch.randn(3, 5, 6, 8, device="cuda")
    ref = f.clone()
    b0 = torch.tensor([1.0, 2.0, 3.0], device="cuda"); b1 = torch.tensor([-1.0, -2.0, -3.0], device="cuda")
    B.dn_apply_bc_per_sample(3, 8, 6, 5, 3, b0, b1, f)
    for b in range(3):
        ref[b, :, :, 0] = b0[b]; ref[b, :, :, -1] = b1[b]
    assert torch.equal(f, ref)
    with pytest.raises(B.DnError) as e:
        B.dn_apply_bc_per_sample(3, 8, 6, 5, 3, b0, None, f)
    assert e.value.status == B.DN_ERR_NULL


def test_cg_and_host_entry_with_per_sample_values():
    bs, n = 3, 24
    inp = inputs.random_inputs(2, n, n, 1, bs, 2, seed=8, f_const=1.0)
    b0 = np.array([1.0, 0.25, -0.5], dtype=np.float32)
    b1 = np.array([0.0, 1.25, 0.5], dtype=np.float32)
    p = B.Problem(dim=2, nx=n, ny=n, nz=1, batch=bs, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=dev(inp.kl_w), f_const=1.0,
                  bc_x0_b=dev(b0), bc_x1_b=dev(b1))
    u = dev(inp.u)
    relres = torch.empty(bs, device="cuda")
    B.dn_cg_solve(p, u, 300, 1e-6, relres, None, B.new_cg_workspace(p))
    torch.cuda.synchronize()
    for b in range(bs):
        pb = oracle.Problem(dim=2, nx=n, ny=n, nz=1, batch=1, nu_mode=oracle.NU_KL_GAUSS, kl_modes=2, kl_w=inp.kl_w[b:b + 1],
                            f_const=1.0, bc_x0=float(b0[b]), bc_x1=float(b1[b]))
        K, F = oracle.assemble(pb)
        us = oracle.solve_dirichlet(pb, K, F)
        assert np.abs(u[b].cpu().numpy() - us).max() <= 2e-4 * np.abs(us).max()
    # host entry point: the per-sample values are host arrays there
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).pin_memory()
    ph = B.Problem(dim=2, nx=n, ny=n, nz=1, batch=bs, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=pin(inp.kl_w), f_const=1.0,
                   flags=B.DN_IMPOSE_BC_ON_LOAD, bc_x0_b=pin(b0), bc_x1_b=pin(b1))
    r_h = torch.empty(bs, n, n).pin_memory(); J_h = torch.empty(bs).pin_memory()
    B.dn_energy_grad_host(ph, pin(inp.u), None, J_h, r_h, B.new_host_staging(ph))
    pd = B.Problem(dim=2, nx=n, ny=n, nz=1, batch=bs, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=dev(inp.kl_w), f_const=1.0,
                   flags=B.DN_IMPOSE_BC_ON_LOAD, bc_x0_b=dev(b0), bc_x1_b=dev(b1))
    J = torch.empty(bs, device="cuda"); r = torch.empty(bs, n, n, device="cuda")
    B.dn_energy_grad(pd, dev(inp.u), None, J, r, B.new_workspace(pd))
    torch.cuda.synchronize()
    # the host entry point runs the batch in chunks, whose blocks may be cut differently: same numbers up to summation order
    assert (r.cpu() - r_h).abs().max() <= 1e-6 * r_h.abs().max() and torch.allclose(J.cpu(), J_h, rtol=1e-6, atol=0.0)
