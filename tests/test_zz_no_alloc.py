"""dn_energy_grad_static -- the entry point for callers that cannot allocate device memory (they pass
inputs and outputs only; the scratch is an array inside the library).  Its results must be those of
dn_energy_grad with a caller-provided workspace, call after call, although all calls share one array.
Collected last so that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs

pytestmark = pytest.mark.gpu


def _run_pair(inp, mode, nu=None, flags=0, f=None):
    w = torch.from_numpy(inp.kl_w).cuda()
    u = torch.from_numpy(inp.u).cuda()
    p = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu,
                  kl_modes=inp.kl_modes, kl_w=w, f_const=inp.f_const, f=f, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1, flags=flags)
    r_ref = torch.empty_like(u); J_ref = torch.empty(inp.batch, device="cuda")
    B.dn_energy_grad(p, u, None, J_ref, r_ref, B.new_workspace(p))
    r = torch.full_like(u, float("nan")); J = torch.full((inp.batch,), float("nan"), device="cuda")
    B.dn_energy_grad_static(p, u, None, J, r)
    torch.cuda.synchronize()
    return J_ref.cpu().numpy(), r_ref.cpu().numpy(), J.cpu().numpy(), r.cpu().numpy()


def test_static_scratch_matches_workspace_entry_point_on_consecutive_calls():
    # two calls in a row with different problems (2D KL, then 3D nodal, then 2D again): the array
    # still holds the previous call's tables and partials each time
    cases = [(inputs.make_inputs(0), B.DN_NU_KL_GAUSS), (inputs.make_inputs(3, samples=range(2)), B.DN_NU_NODAL),
             (inputs.make_inputs(1, samples=range(4)), B.DN_NU_KL_GAUSS), (inputs.make_inputs(0), B.DN_NU_KL_GAUSS),
             # wide 2D rows: the strip kernel when its coefficient table fits the array, else the tiled kernel
             (inputs.random_inputs(2, 1024, 64, 1, 2, 4, seed=9, f_const=0.5), B.DN_NU_KL_GAUSS),
             (inputs.random_inputs(2, 1024, 4000, 1, 6, 6, seed=10), B.DN_NU_KL_GAUSS),
             # rows wider than the tiled kernel takes (2048): the strip kernel, its table within the array
             (inputs.random_inputs(2, 2052, 40, 1, 2, 5, seed=11, f_const=0.25), B.DN_NU_KL_GAUSS),
             (inputs.random_inputs(2, 2052, 40, 1, 2, 5, seed=11, f_const=0.25), B.DN_NU_KL_NODAL),
             (inputs.make_inputs(0), B.DN_NU_KL_GAUSS)]
    for inp, mode in cases:
        nu = None
        if mode == B.DN_NU_NODAL:
            nu = torch.empty(inp.u.shape, device="cuda")
            B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, torch.from_numpy(inp.kl_w).cuda(), nu)
        J_ref, r_ref, J, r = _run_pair(inp, mode, nu)
        assert np.isfinite(J).all() and np.isfinite(r).all()
        assert np.all(np.abs(J - J_ref) <= 1e-5 * np.abs(J_ref))
        assert np.abs(r - r_ref).max() <= 1e-5 * np.abs(r_ref).max()


def test_static_scratch_with_nodal_forcing_when_the_strip_table_does_not_fit():
    """Nodal forcing on a tall grid: the strip kernel's coefficient table (8 x 2100 rows of 64 bytes) exceeds the array,
    and the kernels that take over must still apply the nodal forcing (the any-size kernel does; the tiled ones cannot)."""
    for dim, shape in ((2, (256, 2100, 1)), (3, (64, 64, 70))):
        inp = inputs.random_inputs(dim, *shape, 8, 6 if dim == 2 else 3, seed=21)
        f = torch.from_numpy(inputs.random_field(inp.u.shape, 5, scale=2.0)).cuda()
        J_ref, r_ref, J, r = _run_pair(inp, B.DN_NU_KL_GAUSS, f=f)
        assert np.all(np.abs(J - J_ref) <= 1e-5 * np.abs(J_ref))
        assert np.abs(r - r_ref).max() <= 1e-5 * np.abs(r_ref).max()


def test_static_scratch_refuses_problems_beyond_its_size():
    inp = inputs.random_inputs(3, 130, 130, 130, 4, 2, seed=1)         # any-size kernels: partials exceed 1 MiB
    w = torch.from_numpy(inp.kl_w).cuda(); u = torch.from_numpy(inp.u).cuda()
    p = B.Problem(dim=3, nx=130, ny=130, nz=130, batch=4, kl_modes=2, kl_w=w)
    r = torch.zeros_like(u)
    with pytest.raises(B.DnError) as e:
        B.dn_energy_grad_static(p, u, None, None, r)
    assert e.value.status == B.DN_ERR_WORKSPACE
    assert float(r.abs().max()) == 0.0                                   # nothing was enqueued
    # a wide 2D grid whose strip-kernel table exceeds the array and that no other kernel family serves within 1 MiB
    inp = inputs.random_inputs(2, 4096, 4096, 1, 2, 6, seed=2)
    w = torch.from_numpy(inp.kl_w).cuda(); u = torch.from_numpy(inp.u).cuda()
    p = B.Problem(dim=2, nx=4096, ny=4096, batch=2, kl_modes=6, kl_w=w)
    r = torch.zeros_like(u)
    with pytest.raises(B.DnError) as e:
        B.dn_energy_grad_static(p, u, None, None, r)
    assert e.value.status == B.DN_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert float(r.abs().max()) == 0.0
