"""Plants plausible mistakes in a COPY of the Burgers oracle's source (on the CPU) and checks that a condensed
version of its pins notices each one: a flipped or mis-weighted stencil, a wrong normalisation, the sign of the
convective term, a dropped loss term, a wrong scatter offset or a dropped term of the gradient."""
import os
import types

import numpy as np
import pytest

from oracle import burgers as real

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "burgers.py")

MUTATIONS = {
    "sobel_sign": ("SX = np.array([[-1.0, 0.0, 1.0], [-2.0, 0.0, 2.0], [-1.0, 0.0, 1.0]])",
                   "SX = np.array([[1.0, 0.0, -1.0], [2.0, 0.0, -2.0], [1.0, 0.0, -1.0]])"),
    "sobel_centre_weight": ("[-2.0, 0.0, 2.0]", "[-1.0, 0.0, 1.0]"),
    "t_stencil_not_transposed": ("ST = SX.T.copy()", "ST = SX.copy()"),
    "stencil_operand_transposed": ("ux += SX[dj + 1, di + 1] * blk", "ux += SX[di + 1, dj + 1] * blk"),
    "normalisation": ("return ux / (8.0 * hx), ut / (8.0 * ht)", "return ux / (4.0 * hx), ut / (8.0 * ht)"),
    "x_scaled_by_ht": ("return ux / (8.0 * hx), ut / (8.0 * ht)", "return ux / (8.0 * ht), ut / (8.0 * ht)"),
    "convective_sign_in_loss": ("    res = ut + uc * ux\n", "    res = ut - uc * ux\n"),
    "convective_sign_in_residual": ("return ut + np.asarray(u, dtype=np.float64)[..., 1:-1, 1:-1] * ux",
                                    "return ut - np.asarray(u, dtype=np.float64)[..., 1:-1, 1:-1] * ux"),
    "pde_norm_weight": ("Lp = hx * ht * (res ** 2)", "Lp = hx * (res ** 2)"),
    "inflow_term_dropped": (" + ht * (u[:, :, 0] ** 2).sum(axis=1)", ""),
    "initial_condition_frequency": ("np.cos(2.0 * np.pi * c[:, None] * x[None, :])", "np.cos(np.pi * c[:, None] * x[None, :])"),
    "lambda_not_applied": ("return Lp + lam * Lb, Lp, Lb, g", "return Lp + Lb, Lp, Lb, g"),
    "gradient_centre_term_dropped": ("    g[:, 1:-1, 1:-1] += 2.0 * hx * ht * res * ux\n", ""),
    "gradient_scatter_offset": ("g[:, 1 + dj:nt - 1 + dj, 1 + di:nx - 1 + di] +=", "g[:, 1 - dj:nt - 1 - dj, 1 + di:nx - 1 + di] +="),
    "gradient_x_coefficient": ("+ uc * SX[dj + 1, di + 1] / (8.0 * hx)", "+ SX[dj + 1, di + 1] / (8.0 * hx)"),
    "boundary_gradient_factor": ("g[:, 0, :] += lam * 2.0 * hx * (u[:, 0, :] - u0)", "g[:, 0, :] += lam * hx * (u[:, 0, :] - u0)"),
    "inflow_gradient_dropped": ("    g[:, :, 0] += lam * 2.0 * ht * u[:, :, 0]\n", ""),
    "upstream_gradient_ignored": ("        g *= np.asarray(gL, dtype=np.float64)[:, None, None]\n", "        pass\n"),
}


def load(mutation=None):
    src = open(SRC).read()
    if mutation is not None:
        old, new = MUTATIONS[mutation]
        assert src.count(old) == 1, f"mutation '{mutation}' does not apply to the oracle source"
        src = src.replace(old, new)
    mod = types.ModuleType("burgers_mutant")
    exec(compile(src, SRC, "exec"), mod.__dict__)
    return mod


def pins_hold(ob) -> bool:
    rng = np.random.default_rng(12)
    mesh = lambda nx, nt, T=0.2: (np.arange(nx)[None, :] / (nx - 1), T * np.arange(nt)[:, None] / (nt - 1))
    # derivatives of a field quadratic in x and t
    x, t = mesh(9, 7)
    u = 0.3 - 1.7 * x + 2.5 * t + 0.8 * x * t + 1.1 * x * x - 0.4 * t * t
    ux, ut = ob.derivatives(u[None])
    if not (np.allclose(ux[0], (-1.7 + 0.8 * t + 2.2 * x)[1:-1, 1:-1], atol=1e-11)
            and np.allclose(ut[0], (2.5 + 0.8 * x - 0.8 * t)[1:-1, 1:-1], atol=1e-11)):
        return False
    # loss of a linear field, typed out
    nx, nt, T = 12, 9, 0.2
    x, t = mesh(nx, nt, T)
    a, b, c = 0.2, 0.5, -0.3
    u = (a + b * x + c * t)[None]
    hx, ht = 1.0 / (nx - 1), T / (nt - 1)
    res = c + (a + b * x + c * t) * b
    Lp = hx * ht * (res[1:-1, 1:-1] ** 2).sum()
    u0 = 0.5 * (1 - np.cos(2 * np.pi * 2.3 * x[0]))   # not an integer: whole periods would hide a wrong frequency
    Lb = hx * ((u[0, 0] - u0) ** 2).sum() + ht * (u[0, :, 0] ** 2).sum()
    L, Lp_o, Lb_o, _ = ob.loss_grad(u, np.array([2.3]), T=T, lam=0.7)
    if not (np.isclose(Lp_o[0], Lp, rtol=1e-12) and np.isclose(Lb_o[0], Lb, rtol=1e-12) and np.isclose(L[0], Lp + 0.7 * Lb, rtol=1e-12)):
        return False
    # residual of the exact characteristic solution is O(h^2)
    errs = []
    for n in (33, 65):
        x, t = mesh(n, n, 0.1)
        u = 0.5 * (1 - np.cos(2 * np.pi * x)) * np.ones_like(t)
        for _ in range(200):
            u = 0.5 * (1 - np.cos(2 * np.pi * (x - u * t)))
        errs.append(np.abs(ob.residual(u[None], T=0.1)[0]).max())
    if not (errs[0] < 0.2 and 3.0 < errs[0] / errs[1] < 5.0):
        return False
    # gradient against central differences, with an upstream gradient
    nx, nt = 7, 6
    cpar = np.array([3.3, 5.1])
    u = rng.standard_normal((2, nt, nx))
    gL = np.array([1.5, -0.5])
    g = ob.loss_grad(u, cpar, lam=0.6, gL=gL)[3]
    eps = 1e-5
    for idx in np.ndindex(*u.shape):
        up = u.copy(); up[idx] += eps
        um = u.copy(); um[idx] -= eps
        num = gL[idx[0]] * (ob.loss_grad(up, cpar, lam=0.6)[0][idx[0]] - ob.loss_grad(um, cpar, lam=0.6)[0][idx[0]]) / (2 * eps)
        if abs(num - g[idx]) > 1e-6 * max(1.0, np.abs(g).max()):
            return False
    return True


def test_condensed_pins_hold_for_the_real_oracle():
    assert pins_hold(real) and pins_hold(load())


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_noticed(name):
    assert not pins_hold(load(name)), f"the pins did not notice the planted mistake '{name}'"
