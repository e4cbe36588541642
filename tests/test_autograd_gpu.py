"""The loss as a PyTorch op: its gradient is the residual, and minimising it with L-BFGS (the optimiser the
paper found fastest) reaches the discrete FEM solution that the oracle's dense direct solve gives."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs
from paper_2007_12792_b200.autograd import energy

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dim,n", [(2, 16), (3, 8)])
def test_backward_is_residual_and_lbfgs_reaches_the_direct_solution(dim, n):
    nz = n if dim == 3 else 1
    inp = inputs.random_inputs(dim, n, n, nz, 2, 2, seed=77, f_const=1.0)
    w = torch.from_numpy(inp.kl_w).cuda()
    p = B.Problem(dim=dim, nx=n, ny=n, nz=nz, batch=2, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=w, f_const=1.0)
    po = oracle.Problem(dim=dim, nx=n, ny=n, nz=nz, batch=2, nu_mode=oracle.NU_KL_GAUSS, kl_modes=2, kl_w=inp.kl_w, f_const=1.0)
    u = torch.from_numpy(inp.u).cuda().requires_grad_(True)
    J = energy(u, p)
    (J * torch.tensor([1.0, 3.0], device="cuda")).sum().backward()
    Jo, _, _, ro = oracle.energy_grad(po, inp.u, gJ=np.array([1.0, 3.0]))
    assert np.allclose(J.detach().cpu().numpy(), Jo, rtol=1e-5)
    assert np.abs(u.grad.cpu().numpy() - ro).max() <= 1e-5 * np.abs(ro).max()
    # minimise: Dirichlet nodes get zero gradient, so they keep their boundary values
    x = torch.from_numpy(inp.u).cuda().requires_grad_(True)
    opt = torch.optim.LBFGS([x], lr=1.0, max_iter=400, history_size=30, line_search_fn="strong_wolfe",
                            tolerance_grad=1e-9, tolerance_change=1e-14)

    def closure():
        opt.zero_grad()
        loss = energy(x, p).sum()
        loss.backward()
        return loss

    opt.step(closure)
    Jmin = energy(x, p).detach().cpu().numpy().astype(np.float64)
    for b in range(2):
        pb = oracle.Problem(dim=dim, nx=n, ny=n, nz=nz, batch=1, nu_mode=oracle.NU_KL_GAUSS, kl_modes=2,
                            kl_w=inp.kl_w[b:b + 1], f_const=1.0)
        K, F = oracle.assemble(pb)
        us = oracle.solve_dirichlet(pb, K, F)
        Js = oracle.energy_grad(pb, us[None], want_r=False)[0][0]
        assert Jmin[b] >= Js - 1e-5 * abs(Js)                          # nothing lies below the minimum
        assert abs(Jmin[b] - Js) <= 2e-4 * abs(Js)
        assert np.abs(x.detach().cpu().numpy()[b] - us).max() < 2e-2
