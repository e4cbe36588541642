"""Pins of the fp64 oracle of the paper's Burgers loss (oracle/burgers.py) against closed forms, an exact
solution of the PDE, and finite differences (no GPU)."""
import numpy as np
import pytest

from oracle import burgers as ob

RNG = np.random.default_rng(2007)


def mesh(nx, nt, T=0.2):
    x = np.arange(nx) / (nx - 1)
    t = T * np.arange(nt) / (nt - 1)
    return x[None, :], t[:, None]


@pytest.mark.parametrize("nx,nt", [(9, 7), (16, 33)])
def test_sobel_is_exact_on_low_order_fields(nx, nt):
    x, t = mesh(nx, nt)
    a, b, c = 0.3, -1.7, 2.5
    u = a + b * x + c * t + 0.8 * x * t + 1.1 * x * x - 0.4 * t * t       # quadratic per variable: central differences exact
    ux, ut = ob.derivatives(u[None])
    # u_xx and u_tt are constant, so the (1,2,1) smoothing of the central differences reproduces them exactly
    assert np.allclose(ux[0], (b + 0.8 * t + 2.2 * x)[1:-1, 1:-1], atol=1e-12)
    assert np.allclose(ut[0], (c + 0.8 * x - 0.8 * t)[1:-1, 1:-1], atol=1e-12)


def test_loss_of_a_linear_field_closed_form():
    nx, nt, T = 12, 9, 0.2
    x, t = mesh(nx, nt, T)
    a, b, c = 0.2, 0.5, -0.3
    u = (a + b * x + c * t)[None]
    hx, ht = 1.0 / (nx - 1), T / (nt - 1)
    res = c + (a + b * x + c * t) * b                                      # u_t + u u_x typed out
    Lp = hx * ht * (res[1:-1, 1:-1] ** 2).sum()
    cpar = np.array([2.3])                                                 # not an integer: sums over whole periods would hide a wrong frequency
    u0 = 0.5 * (1 - np.cos(2 * np.pi * 2.3 * x[0]))
    Lb = hx * ((u[0, 0] - u0) ** 2).sum() + ht * (u[0, :, 0] ** 2).sum()
    L, Lp_o, Lb_o, g = ob.loss_grad(u, cpar, T=T, lam=0.7)
    assert Lp_o[0] == pytest.approx(Lp, rel=1e-13) and Lb_o[0] == pytest.approx(Lb, rel=1e-13)
    assert L[0] == pytest.approx(Lp + 0.7 * Lb, rel=1e-13)


def test_residual_of_the_exact_solution_converges_at_second_order():
    """Before the shock the solution is u = u0(x - u t) (characteristics).  Its discrete residual is O(h^2);
    with the wrong sign of the convective term it would be O(1)."""
    c, T = 1.0, 0.1                                                        # shock forms at t = 1/(pi c) > T
    errs = []
    for n in (33, 65, 129):
        x, t = mesh(n, n, T)
        u = 0.5 * (1 - np.cos(2 * np.pi * c * x)) * np.ones_like(t)
        for _ in range(200):                                               # fixed point of u = u0(x - u t)
            u = 0.5 * (1 - np.cos(2 * np.pi * c * (x - u * t)))
        r = ob.residual(u[None], T=T)[0]
        errs.append(np.abs(r).max())
    assert errs[0] < 0.2 and 3.0 < errs[0] / errs[1] < 5.0 and 3.0 < errs[1] / errs[2] < 5.0, errs
    x, t = mesh(65, 65, T)
    wrong = ob.derivatives(u[None], T=T)
    assert np.abs(wrong[1][0] - u[1:-1, 1:-1] * wrong[0][0]).max() > 0.5    # u_t - u u_x is not small


def test_boundary_term_vanishes_on_matching_data_and_is_local():
    nx, nt = 17, 11
    c = np.array([3.0, 4.5])
    u = RNG.standard_normal((2, nt, nx))
    u[:, 0, :] = ob.initial_condition(nx, c)
    u[:, :, 0] = 0.0
    Lb = ob.loss_grad(u, c)[2]
    assert np.all(np.abs(Lb) < 1e-28)
    u2 = u.copy(); u2[1, 0, 5] += 0.25
    hx = 1.0 / (nx - 1)
    assert ob.loss_grad(u2, c)[2][1] == pytest.approx(hx * 0.25 ** 2, rel=1e-12)
    u3 = u.copy(); u3[0, 4, 0] = 0.5
    assert ob.loss_grad(u3, c)[2][0] == pytest.approx((0.2 / (nt - 1)) * 0.25, rel=1e-12)


@pytest.mark.parametrize("nx,nt", [(8, 8), (11, 6)])
def test_gradient_matches_central_differences(nx, nt):
    c = np.array([3.3, 5.1])
    u = RNG.standard_normal((2, nt, nx))
    gL = np.array([1.5, -0.5])
    L, _, _, g = ob.loss_grad(u, c, lam=0.6, gL=gL)
    eps = 1e-5
    num = np.zeros_like(u)
    for idx in np.ndindex(*u.shape):
        up = u.copy(); up[idx] += eps
        um = u.copy(); um[idx] -= eps
        num[idx] = gL[idx[0]] * (ob.loss_grad(up, c, lam=0.6)[0][idx[0]] - ob.loss_grad(um, c, lam=0.6)[0][idx[0]]) / (2 * eps)
    assert np.abs(num - g).max() < 1e-6 * max(1.0, np.abs(g).max())       # L is quartic in u: O(eps^2) truncation


def test_input_recipe_is_reproducible():
    from paper_2007_12792_b200 import inputs
    a = inputs.burgers_inputs(32, 16, 4)
    b = inputs.burgers_inputs(32, 16, 4, samples=[2])
    assert np.array_equal(a.u[2], b.u[0]) and a.c[2] == b.c[0] and 3.0 <= a.c.min() and a.c.max() <= 6.0
