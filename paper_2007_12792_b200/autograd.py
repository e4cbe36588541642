"""The physics loss as a differentiable PyTorch op: forward = per-sample energies J from the fused
CUDA kernel, backward = the residual the same kernel produced (the loss gradient that enters the
generator's back-propagation in Algorithm 1).  No autograd graph is built inside; there is no CPU path."""
from __future__ import annotations

import torch

from . import binding as B


class _Energy(torch.autograd.Function):
    @staticmethod
    def forward(ctx, u, problem, workspace):
        u = u.contiguous()
        J = torch.empty(problem.batch, dtype=torch.float32, device=u.device)
        r = torch.empty_like(u)
        B.dn_energy_grad(problem, u, None, J, r, workspace)
        ctx.save_for_backward(r)
        return J

    @staticmethod
    def backward(ctx, grad_J):
        (r,) = ctx.saved_tensors
        shape = (-1,) + (1,) * (r.dim() - 1)
        return grad_J.reshape(shape).to(r.dtype) * r, None, None


def energy(u: torch.Tensor, problem: B.Problem, workspace: torch.Tensor = None) -> torch.Tensor:
    """J[b] for a batch of fields u (contiguous float32 CUDA tensor); differentiable with respect to u.
    The gradient is the masked residual K(nu) u - F, so Dirichlet nodes receive zero gradient."""
    if workspace is None:
        workspace = B.new_workspace(problem)
    return _Energy.apply(u, problem, workspace)


class _BurgersLoss(torch.autograd.Function):
    @staticmethod
    def forward(ctx, u, problem, workspace):
        u = u.contiguous()
        L = torch.empty(problem.batch, dtype=torch.float32, device=u.device)
        g = torch.empty_like(u)
        B.dn_burgers_loss_grad(problem, u, None, L, None, g, workspace)
        ctx.save_for_backward(g)
        return L

    @staticmethod
    def backward(ctx, grad_L):
        (g,) = ctx.saved_tensors
        return grad_L.reshape(-1, 1, 1).to(g.dtype) * g, None, None


def burgers_loss(u: torch.Tensor, problem: B.Burgers, workspace: torch.Tensor = None) -> torch.Tensor:
    """L[b] = L_p + lambda L_b of the Burgers finite-difference loss for a batch of fields u [B][nt][nx]
    (contiguous float32 CUDA tensor); differentiable with respect to u."""
    if workspace is None:
        workspace = B.new_burgers_workspace(problem)
    return _BurgersLoss.apply(u, problem, workspace)
