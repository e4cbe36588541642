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


def test_burgers_loss_backward_matches_oracle_gradient():
    from oracle import burgers as ob
    from paper_2007_12792_b200.autograd import burgers_loss
    inp = inputs.burgers_inputs(64, 40, 3)
    T32 = float(np.float32(0.2))
    p = B.Burgers(nx=64, nt=40, batch=3, c=torch.from_numpy(inp.c).cuda(), T=T32, lam=0.5)
    u = torch.from_numpy(inp.u).cuda().requires_grad_(True)
    wts = np.array([1.0, -2.0, 0.5])
    (burgers_loss(u, p) * torch.tensor(wts, device="cuda", dtype=torch.float32)).sum().backward()
    go = ob.loss_grad(inp.u, inp.c.astype(np.float64), T=T32, lam=0.5, gL=wts)[3]
    assert np.abs(u.grad.cpu().numpy() - go).max() <= 1e-5 * np.abs(go).max()


class _TinyGenerator(torch.nn.Module):
    """A small convolutional generator (outside the library): latent -> full field, as in the paper's DiffNet."""

    def __init__(self, n, out_scale=1.0):
        super().__init__()
        self.n = n
        self.fc = torch.nn.Linear(4, 8 * (n // 4) * (n // 4))
        self.net = torch.nn.Sequential(
            torch.nn.Upsample(scale_factor=2, mode="bilinear", align_corners=False), torch.nn.Conv2d(8, 8, 3, padding=1),
            torch.nn.Tanh(),
            torch.nn.Upsample(scale_factor=2, mode="bilinear", align_corners=False), torch.nn.Conv2d(8, 1, 3, padding=1))
        self.out_scale = out_scale

    def forward(self, z):
        h = self.fc(z).view(-1, 8, self.n // 4, self.n // 4)
        return self.out_scale * self.net(h)[:, 0]


def test_generator_trained_on_the_energy_alone_approaches_the_fem_minimum():
    """Algorithm 1 in miniature: a generator maps a code of the sampled diffusivity to a field, the only training
    signal is the physics loss; after Adam steps the mean energy has dropped most of the way to the FEM minimum."""
    torch.manual_seed(0)
    n, bs = 32, 4
    inp = inputs.random_inputs(2, n, n, 1, bs, 2, seed=5, f_const=0.0)
    w = torch.from_numpy(inp.kl_w).cuda()
    p = B.Problem(dim=2, nx=n, ny=n, nz=1, batch=bs, nu_mode=B.DN_NU_KL_GAUSS, kl_modes=2, kl_w=w, f_const=0.0,
                  bc_x0=1.0, bc_x1=0.0, flags=B.DN_IMPOSE_BC_ON_LOAD)
    gen = _TinyGenerator(n).cuda()
    opt = torch.optim.Adam(gen.parameters(), lr=3e-3)
    ws = B.new_workspace(p)
    z = w.reshape(bs, -1)
    hist = []
    for _ in range(300):
        opt.zero_grad()
        loss = energy(gen(z).contiguous(), p, ws).mean()
        loss.backward()
        opt.step()
        hist.append(float(loss.detach()))
    Jmin = []
    for b in range(bs):
        pb = oracle.Problem(dim=2, nx=n, ny=n, nz=1, batch=1, nu_mode=oracle.NU_KL_GAUSS, kl_modes=2,
                            kl_w=inp.kl_w[b:b + 1], f_const=0.0, bc_x0=1.0, bc_x1=0.0)
        K, F = oracle.assemble(pb)
        us = oracle.solve_dirichlet(pb, K, F)
        Jmin.append(oracle.energy_grad(pb, us[None], want_r=False)[0][0])
    Jstar = float(np.mean(Jmin))
    assert hist[-1] < hist[0] and hist[-1] >= Jstar - 1e-4 * abs(Jstar)
    assert hist[-1] - Jstar < 0.1 * (hist[0] - Jstar), (hist[0], hist[-1], Jstar)


def test_generator_trained_on_the_burgers_loss_alone_reduces_it():
    from paper_2007_12792_b200.autograd import burgers_loss
    torch.manual_seed(0)
    n, bs = 32, 4
    c = torch.tensor([3.0, 4.0, 5.0, 6.0], device="cuda")
    p = B.Burgers(nx=n, nt=n, batch=bs, c=c, T=float(np.float32(0.2)), lam=1.0)
    gen = _TinyGenerator(n).cuda()
    opt = torch.optim.Adam(gen.parameters(), lr=3e-3)
    ws = B.new_burgers_workspace(p)
    z = torch.stack([c, c * c / 6, torch.ones_like(c), torch.zeros_like(c)], dim=1) / 6
    hist = []
    for _ in range(300):
        opt.zero_grad()
        loss = burgers_loss(gen(z).contiguous(), p, ws).mean()
        loss.backward()
        opt.step()
        hist.append(float(loss.detach()))
    assert np.isfinite(hist).all() and hist[-1] < 0.5 * hist[0], (hist[0], hist[-1])
