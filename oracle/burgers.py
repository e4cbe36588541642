"""TEST INFRASTRUCTURE -- not part of the product.

Plain fp64 statement (numpy) of the paper's own loss for the inviscid Burgers equation
("Introduction", Eq. (Inviscid_Burgers) and Eq. (initial-condition); "DiffNets", Eq. (diffnetloss),
Eq. (pde_loss), Eq. (boundaryloss); "Implementing the forward model": first derivatives by 3x3 Sobel
kernels, x and t operators scaled separately):

    field      u[b][j][i] on x_i = i hx, t_j = j ht,  hx = 1/(nx-1), ht = T/(nt-1), T = 0.2
    u_x(i,j)   = sum_{dj,di} Sx[dj][di] u[j+dj][i+di] / (8 hx),  Sx = [[-1,0,1],[-2,0,2],[-1,0,1]]
    u_t(i,j)   = sum_{dj,di} St[dj][di] u[j+dj][i+di] / (8 ht),  St = Sx transposed
    res(i,j)   = u_t + u u_x                        at interior nodes 0 < i < nx-1, 0 < j < nt-1
    L_p[b]     = hx ht sum_interior res^2
    L_b[b]     = hx sum_i (u[0][i] - u0(x_i; c_b))^2 + ht sum_j u[j][0]^2,   u0 = (1 - cos(2 pi c x)) / 2
    L[b]       = L_p[b] + lam L_b[b],      g = dL/du   (every node)

The paper gives the stencils by name only; the normalisations (exact on linear fields), the discrete
norms and the inflow-only boundary term (u >= 0, so characteristics enter through x = 0) are this
build's readings.  Pins: tests/test_burgers_pins.py.
"""
from __future__ import annotations

import numpy as np

SX = np.array([[-1.0, 0.0, 1.0], [-2.0, 0.0, 2.0], [-1.0, 0.0, 1.0]])   # [dj+1][di+1]
ST = SX.T.copy()


def grid(nx: int, nt: int, T: float = 0.2):
    return 1.0 / (nx - 1), T / (nt - 1)


def initial_condition(nx: int, c) -> np.ndarray:
    x = np.arange(nx) / (nx - 1)
    c = np.atleast_1d(np.asarray(c, dtype=np.float64))
    return 0.5 * (1.0 - np.cos(2.0 * np.pi * c[:, None] * x[None, :]))


def derivatives(u: np.ndarray, T: float = 0.2):
    """(u_x, u_t) at the interior nodes, shape [B][nt-2][nx-2]."""
    u = np.asarray(u, dtype=np.float64)
    nt, nx = u.shape[-2:]
    hx, ht = grid(nx, nt, T)
    ux = np.zeros(u.shape[:-2] + (nt - 2, nx - 2))
    ut = np.zeros_like(ux)
    for dj in (-1, 0, 1):
        for di in (-1, 0, 1):
            blk = u[..., 1 + dj:nt - 1 + dj, 1 + di:nx - 1 + di]
            ux += SX[dj + 1, di + 1] * blk
            ut += ST[dj + 1, di + 1] * blk
    return ux / (8.0 * hx), ut / (8.0 * ht)


def residual(u: np.ndarray, T: float = 0.2) -> np.ndarray:
    ux, ut = derivatives(u, T)
    return ut + np.asarray(u, dtype=np.float64)[..., 1:-1, 1:-1] * ux


def loss_grad(u: np.ndarray, c, T: float = 0.2, lam: float = 1.0, gL=None):
    """Returns (L[B], Lp[B], Lb[B], g[B][nt][nx]); g is multiplied by gL[b] when given."""
    u = np.asarray(u, dtype=np.float64)
    B, nt, nx = u.shape
    hx, ht = grid(nx, nt, T)
    ux, ut = derivatives(u, T)
    uc = u[:, 1:-1, 1:-1]
    res = ut + uc * ux
    Lp = hx * ht * (res ** 2).sum(axis=(1, 2))
    u0 = initial_condition(nx, c)
    Lb = hx * ((u[:, 0, :] - u0) ** 2).sum(axis=1) + ht * (u[:, :, 0] ** 2).sum(axis=1)
    g = np.zeros_like(u)
    # d res(i,j) / d u[j+dj][i+di] = St/(8 ht) + u(i,j) Sx/(8 hx), plus u_x at the centre
    for dj in (-1, 0, 1):
        for di in (-1, 0, 1):
            coef = ST[dj + 1, di + 1] / (8.0 * ht) + uc * SX[dj + 1, di + 1] / (8.0 * hx)
            g[:, 1 + dj:nt - 1 + dj, 1 + di:nx - 1 + di] += 2.0 * hx * ht * res * coef
    g[:, 1:-1, 1:-1] += 2.0 * hx * ht * res * ux
    g[:, 0, :] += lam * 2.0 * hx * (u[:, 0, :] - u0)
    g[:, :, 0] += lam * 2.0 * ht * u[:, :, 0]
    if gL is not None:
        g *= np.asarray(gL, dtype=np.float64)[:, None, None]
    return Lp + lam * Lb, Lp, Lb, g
