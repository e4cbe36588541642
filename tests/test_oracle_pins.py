"""Pins of the fp64 CPU oracle against what the mathematics fixes (no GPU).

Every check compares the oracle with something that is not the oracle: closed
forms, textbook element matrices (tests/golden), tensor-product assembly from
1-D matrices, adaptive quadrature from scipy, finite differences, a dense solve.
"""
import os

import numpy as np
import pytest

import oracle
from oracle import Problem, NU_NODAL, NU_KL_GAUSS, NU_KL_NODAL, NO_MASK, IMPOSE_BC_ON_LOAD
from paper_2007_12792_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(20071279)


def lin_profile(shape):
    nx = shape[-1]
    return np.broadcast_to(1.0 - np.arange(nx) / (nx - 1), shape).astype(np.float64).copy()


def trapezoid_weights(dim, nx, ny, nz):
    def w1(n):
        w = np.full(n, 1.0 / (n - 1)); w[0] *= 0.5; w[-1] *= 0.5
        return w
    if dim == 2:
        return w1(ny)[:, None] * w1(nx)[None, :]
    return w1(nz)[:, None, None] * w1(ny)[None, :, None] * w1(nx)[None, None, :]


def const_nu(p, c):
    return np.full(p.shape, c, dtype=np.float32)


GRIDS = [(2, 9, 9, 1), (2, 12, 7, 1), (3, 5, 5, 5), (3, 6, 4, 5)]


# ---- P1 / P2: linear profile, constant nu ------------------------------------------------
@pytest.mark.parametrize("dim,nx,ny,nz", GRIDS)
def test_linear_profile_energy_and_residual(dim, nx, ny, nz):
    c = 2.5
    p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, flags=NO_MASK)
    p.nu = const_nu(p, c)
    u = lin_profile(p.shape)
    J, Jd, Jl, r = oracle.energy_grad(p, u)
    assert J[0] == pytest.approx(c / 2, rel=1e-13)
    assert np.abs(r[..., 1:-1]).max() < 1e-13            # every non-Dirichlet node, also on zero-flux faces
    assert r[..., 0].sum() == pytest.approx(+c, rel=1e-12)   # reaction on x = 0 (flux nu*1 leaves through it)
    assert r[..., -1].sum() == pytest.approx(-c, rel=1e-12)
    p.flags = 0
    r_masked = oracle.energy_grad(p, u)[3]
    assert np.all(r_masked[..., 0] == 0.0) and np.all(r_masked[..., -1] == 0.0)


# ---- P6: textbook element matrices and stencils -------------------------------------------
def test_square_element_matrix_golden():
    gold = np.loadtxt(os.path.join(GOLD, "q1_square_stiffness.txt"))
    for nu in (1.0, 3.0):
        p = Problem(dim=2, nx=2, ny=2, batch=1, nu_mode=NU_NODAL)
        p.nu = const_nu(p, nu)
        K, F = oracle.assemble(p)
        assert np.allclose(K, nu * gold, atol=1e-14)


def test_cube_element_matrix_golden():
    vals = np.loadtxt(os.path.join(GOLD, "q1_cube_stiffness.txt"))
    p = Problem(dim=3, nx=2, ny=2, nz=2, batch=1, nu_mode=NU_NODAL)
    p.nu = const_nu(p, 1.0)
    K, _ = oracle.assemble(p)
    for a in range(8):
        for b in range(8):
            assert K[a, b] == pytest.approx(vals[bin(a ^ b).count("1")], abs=1e-14)


def test_interior_stencils_golden():
    with open(os.path.join(GOLD, "q1_interior_stencils.txt")) as fh:
        rows = [np.array(l.split(), dtype=float) for l in fh if l.strip() and not l.startswith("#")]
    n = 5
    p = Problem(dim=2, nx=n, ny=n, batch=1, nu_mode=NU_NODAL); p.nu = const_nu(p, 1.0)
    K, _ = oracle.assemble(p)
    c = 2 * n + 2
    row = K[c].reshape(n, n)
    assert row[2, 2] == pytest.approx(rows[0][0], rel=1e-13)
    nb = [row[2 + dy, 2 + dx] for dy in (-1, 0, 1) for dx in (-1, 0, 1) if (dx, dy) != (0, 0)]
    assert np.allclose(nb, rows[0][1], rtol=1e-13)
    assert np.count_nonzero(np.abs(row) > 1e-15) == 9
    p = Problem(dim=3, nx=n, ny=n, nz=n, batch=1, nu_mode=NU_NODAL); p.nu = const_nu(p, 1.0)
    K, _ = oracle.assemble(p)
    h = 1.0 / (n - 1)
    row = K[(2 * n + 2) * n + 2].reshape(n, n, n)
    for dz in (-1, 0, 1):
        for dy in (-1, 0, 1):
            for dx in (-1, 0, 1):
                k = abs(dx) + abs(dy) + abs(dz)
                assert row[2 + dz, 2 + dy, 2 + dx] == pytest.approx(rows[1][k] * h, abs=1e-14)


def _k1d(n):
    h = 1.0 / (n - 1)
    S = np.zeros((n, n)); M = np.zeros((n, n))
    for e in range(n - 1):
        S[e:e + 2, e:e + 2] += np.array([[1, -1], [-1, 1]]) / h
        M[e:e + 2, e:e + 2] += h * np.array([[2, 1], [1, 2]]) / 6
    return S, M


@pytest.mark.parametrize("dim,nx,ny,nz", GRIDS)
def test_dense_assembly_equals_tensor_product_of_1d_matrices(dim, nx, ny, nz):
    """Constant nu, rectangular cells (hx != hy): K = sum over axes of kron(M,..,S,..,M); F = f * kron of M 1."""
    nu, f = 1.7, 0.8
    p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, f_const=f); p.nu = const_nu(p, nu)
    K, F = oracle.assemble(p)
    Sx, Mx = _k1d(nx); Sy, My = _k1d(ny)
    if dim == 2:
        Kref = np.kron(My, Sx) + np.kron(Sy, Mx)
        Fref = f * np.kron(My.sum(1), Mx.sum(1))
    else:
        Sz, Mz = _k1d(nz)
        Kref = np.kron(Mz, np.kron(My, Sx)) + np.kron(Mz, np.kron(Sy, Mx)) + np.kron(Sz, np.kron(My, Mx))
        Fref = f * np.kron(Mz.sum(1), np.kron(My.sum(1), Mx.sum(1)))
    assert np.allclose(K, nu * Kref, atol=1e-12)
    assert np.allclose(F, Fref, atol=1e-14)
    # and the matrix-free residual is K u - F for that matrix
    u = RNG.standard_normal(p.shape)
    p.flags = NO_MASK
    r = oracle.energy_grad(p, u)[3]
    assert np.allclose(r.ravel(), nu * Kref @ u.ravel() - Fref, atol=1e-11)


# ---- P3 / P4: J is quadratic; gradient = finite differences ---------------------------------
def _problem(dim, nx, ny, nz, mode, batch=1, m=2, f_const=0.7, seed=5):
    p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=batch, nu_mode=mode, f_const=f_const, flags=NO_MASK)
    if mode == NU_NODAL:
        p.nu = inputs.random_positive_field(p.shape, seed)
    else:
        p.kl_modes = m
        p.kl_w = np.stack([inputs.draw_weights(np.random.default_rng(seed + b), dim, m) for b in range(batch)])
    return p


@pytest.mark.parametrize("mode", [NU_NODAL, NU_KL_GAUSS, NU_KL_NODAL])
@pytest.mark.parametrize("dim,nx,ny,nz", [(2, 8, 8, 1), (3, 5, 5, 5), (2, 7, 5, 1)])
def test_quadratic_in_t_and_finite_differences(mode, dim, nx, ny, nz):
    p = _problem(dim, nx, ny, nz, mode)
    u = RNG.standard_normal(p.shape)
    v = RNG.standard_normal(p.shape)
    J0, _, _, r = oracle.energy_grad(p, u)
    ts = np.array([-2.0, -1.0, 0.0, 1.0, 2.0])
    Js = np.array([oracle.energy_grad(p, u + t * v, want_r=False)[0][0] for t in ts])
    d3 = np.diff(Js, 3)
    assert np.abs(d3).max() < 1e-10 * np.abs(Js).max()          # third differences vanish
    slope = (Js[3] - Js[1]) / 2.0                                   # exact for a quadratic
    assert slope == pytest.approx(np.vdot(r, v), rel=1e-11, abs=1e-11)
    K, F = oracle.assemble(p)
    assert np.diff(Js, 2)[1] == pytest.approx(v.ravel() @ K @ v.ravel(), rel=1e-10)
    # central differences node by node
    eps = 1e-3
    g = np.zeros(u.size)
    for i in range(u.size):
        e = np.zeros(u.size); e[i] = eps
        e = e.reshape(u.shape)
        g[i] = (oracle.energy_grad(p, u + e, want_r=False)[0][0] - oracle.energy_grad(p, u - e, want_r=False)[0][0]) / (2 * eps)
    assert np.abs(g - r.ravel()).max() < 1e-9 * max(1.0, np.abs(r).max())


# ---- P5: residual vanishes at the discrete solution -------------------------------------------
@pytest.mark.parametrize("mode", [NU_NODAL, NU_KL_GAUSS, NU_KL_NODAL])
@pytest.mark.parametrize("dim,nx,ny,nz", [(2, 6, 6, 1), (2, 9, 5, 1), (3, 4, 4, 4), (3, 5, 4, 3)])
def test_residual_zero_at_direct_solution(mode, dim, nx, ny, nz):
    p = _problem(dim, nx, ny, nz, mode, f_const=1.0)
    p.bc_x0, p.bc_x1 = 1.0, 0.0
    K, F = oracle.assemble(p)
    us = oracle.solve_dirichlet(p, K, F)[None]
    # independent check of the solver itself
    free = np.ones(p.shape[1:], bool); free[..., 0] = False; free[..., -1] = False
    fi = np.flatnonzero(free.ravel()); di = np.flatnonzero(~free.ravel())
    uref = us.ravel().copy()
    uref[fi] = np.linalg.solve(K[np.ix_(fi, fi)], F[fi] - K[np.ix_(fi, di)] @ uref[di])
    assert np.allclose(us.ravel(), uref, atol=1e-12)
    assert np.all(us[..., 0] == 1.0) and np.all(us[..., -1] == 0.0)
    p.flags = 0
    J, _, _, r = oracle.energy_grad(p, us)
    assert np.abs(r).max() < 1e-12
    # the solution minimises J among fields with the same boundary values
    w = RNG.standard_normal(p.shape); w[..., 0] = 0; w[..., -1] = 0
    assert oracle.energy_grad(p, us + 0.1 * w, want_r=False)[0][0] > J[0]


# ---- P7 / P8 / P12: partition of unity, Euler identity, symmetry ------------------------------
@pytest.mark.parametrize("mode", [NU_NODAL, NU_KL_GAUSS, NU_KL_NODAL])
@pytest.mark.parametrize("dim,nx,ny,nz", GRIDS)
def test_partition_of_unity_euler_symmetry(mode, dim, nx, ny, nz):
    p = _problem(dim, nx, ny, nz, mode, batch=2, f_const=0.9)
    u = RNG.standard_normal(p.shape)
    J, Jd, Jl, r = oracle.energy_grad(p, u)
    for b in range(2):
        assert r[b].sum() == pytest.approx(-0.9, rel=1e-11)                    # sum_i (Ku)_i = 0, sum_i F_i = f |Omega|
        assert np.vdot(u[b], r[b]) == pytest.approx(2 * Jd[b] - Jl[b], rel=1e-11)   # <u, Ku - F> = 2 Jdiff - Jload
        assert Jd[b] > 0 and J[b] == pytest.approx(Jd[b] - Jl[b], rel=1e-14)
    # nodal forcing: F_i = (M f)_i, so sum_i F_i = integral of the interpolant = trapezoid rule
    p.f = inputs.random_field(p.shape, 3)
    r2 = oracle.energy_grad(p, u)[3]
    tw = trapezoid_weights(dim, nx, ny, nz)
    for b in range(2):
        assert r2[b].sum() == pytest.approx(-(tw * p.f[b].astype(np.float64)).sum(), rel=1e-10, abs=1e-12)
    # symmetry: <v, K w> = <w, K v> with K z = r(z) - r(0)
    p.f = None
    v = RNG.standard_normal(p.shape); w = RNG.standard_normal(p.shape)
    r0 = oracle.energy_grad(p, np.zeros(p.shape))[3]
    Kv = oracle.energy_grad(p, v)[3] - r0
    Kw = oracle.energy_grad(p, w)[3] - r0
    assert np.vdot(w, Kv) == pytest.approx(np.vdot(v, Kw), rel=1e-11)
    K, _ = oracle.assemble(p, b=1)
    assert np.allclose(K, K.T, atol=1e-13)
    assert np.allclose(K.sum(1), 0.0, atol=1e-12)
    assert np.linalg.eigvalsh(K).min() > -1e-12


# ---- P9: constant field, unit forcing ---------------------------------------------------------
@pytest.mark.parametrize("dim,nx,ny,nz", GRIDS)
def test_constant_field_unit_forcing(dim, nx, ny, nz):
    c0 = 0.37
    p = _problem(dim, nx, ny, nz, NU_KL_GAUSS, f_const=1.0)
    u = np.full(p.shape, c0)
    J, Jd, Jl, r = oracle.energy_grad(p, u)
    assert J[0] == pytest.approx(-c0, rel=1e-13) and abs(Jd[0]) < 1e-25
    assert np.allclose(r[0], -trapezoid_weights(dim, nx, ny, nz), atol=1e-15)


# ---- P10 / P11: nodal mode is integrated exactly by the 2-point rule ---------------------------
@pytest.mark.parametrize("dim,nx,ny,nz", GRIDS)
def test_nodal_mode_trapezoid_energy_and_three_point_rule(dim, nx, ny, nz):
    p = _problem(dim, nx, ny, nz, NU_NODAL, f_const=0.0)
    u = lin_profile(p.shape)
    J = oracle.energy_grad(p, u, want_r=False)[0][0]
    tw = trapezoid_weights(dim, nx, ny, nz)
    assert J == pytest.approx(0.5 * (tw * p.nu[0].astype(np.float64)).sum(), rel=1e-13)
    # general u, nodal forcing: 3-point rule gives the same numbers
    u = RNG.standard_normal(p.shape); p.f = inputs.random_field(p.shape, 9)
    a = oracle.energy_grad(p, u)
    p.nquad = 3
    b = oracle.energy_grad(p, u)
    assert a[0][0] == pytest.approx(b[0][0], rel=1e-12)
    assert np.abs(a[3] - b[3]).max() < 1e-12 * np.abs(a[3]).max()


def test_single_element_interpolated_nodal_nu_closed_form():
    """One element, u = x y (z): the integrand nu |grad u|^2 is a polynomial, integrated by hand from 1-D moments
    int (1-t) dt = int t dt = 1/2,  int (1-t) t^2 dt = 1/12,  int t^3 dt = 1/4.  Fails if nu is not interpolated to
    the Gauss points (an element-mean nu gives a different number)."""
    m0 = {0: 0.5, 1: 0.5}            # int w_i(t) dt
    m2 = {0: 1.0 / 12.0, 1: 0.25}    # int w_i(t) t^2 dt
    rng = np.random.default_rng(12)
    nu = rng.uniform(0.5, 3.0, (1, 2, 2)).astype(np.float32)
    u = np.array([[[0.0, 0.0], [0.0, 1.0]]])                       # u = x y at the corners
    ref = 0.5 * sum(float(nu[0, j, i]) * (m0[i] * m2[j] + m2[i] * m0[j]) for i in (0, 1) for j in (0, 1))
    p = Problem(dim=2, nx=2, ny=2, batch=1, nu_mode=NU_NODAL, nu=nu)
    assert oracle.energy_grad(p, u, want_r=False)[0][0] == pytest.approx(ref, rel=1e-14)
    nu3 = rng.uniform(0.5, 3.0, (1, 2, 2, 2)).astype(np.float32)
    u3 = np.zeros((1, 2, 2, 2)); u3[0, 1, 1, 1] = 1.0             # u = x y z
    ref3 = 0.5 * sum(float(nu3[0, k, j, i]) * (m0[i] * m2[j] * m2[k] + m2[i] * m0[j] * m2[k] + m2[i] * m2[j] * m0[k])
                     for i in (0, 1) for j in (0, 1) for k in (0, 1))
    p3 = Problem(dim=3, nx=2, ny=2, nz=2, batch=1, nu_mode=NU_NODAL, nu=nu3)
    assert oracle.energy_grad(p3, u3, want_r=False)[0][0] == pytest.approx(ref3, rel=1e-14)


# ---- P13 + KL-at-Gauss position pins ------------------------------------------------------------
def test_kl_field_closed_forms():
    nx, ny = 9, 6
    x = np.arange(nx) / (nx - 1); y = np.arange(ny) / (ny - 1)
    w = np.zeros((1, 3, 3), np.float32)
    assert np.all(oracle.kl_field(2, nx, ny, 1, 1, 3, w) == 1.0)
    w[0, 0, 1] = 1.25                                                    # i = 1 (x), j = 2 (y): denominator 1+1+4
    ref = np.exp(1.25 * np.cos(np.pi * x)[None, :] * np.cos(2 * np.pi * y)[:, None] / 6.0)
    assert np.allclose(oracle.kl_field(2, nx, ny, 1, 1, 3, w)[0], ref, rtol=1e-14)
    w = inputs.draw_weights(np.random.default_rng(1), 2, 3)[None]
    nu = oracle.kl_field(2, nx, ny, 1, 1, 3, w)
    ii = np.arange(1, 4)
    assert nu[0, 0, 0] == pytest.approx(np.exp((w[0].astype(np.float64) / (1 + ii[:, None] ** 2 + ii[None, :] ** 2)).sum()), rel=1e-14)
    assert np.all(nu > 0)
    nz = 5
    z = np.arange(nz) / (nz - 1)
    w3 = np.zeros((2, 3, 3, 3), np.float32); w3[1, 0, 1, 2] = -0.8        # i=1 (x), j=2 (y), k=3 (z): 1+1+4+9
    ref = np.exp(-0.8 * np.cos(np.pi * x)[None, None, :] * np.cos(2 * np.pi * y)[None, :, None]
                 * np.cos(3 * np.pi * z)[:, None, None] / 15.0)
    out = oracle.kl_field(3, nx, ny, nz, 2, 3, w3)
    assert np.all(out[0] == 1.0) and np.allclose(out[1], ref, rtol=1e-14)


def test_kl_nodal_mode_closed_form_and_equivalence():
    """KL evaluated at the nodes, then Q1-interpolated: for u = 1 - x the energy is the trapezoid sum of the
    typed-out KL formula at the nodes; for general u it equals nodal mode fed with that field."""
    for dim, nx, ny, nz in GRIDS:
        w = inputs.draw_weights(np.random.default_rng(21), dim, 2)[None]
        wd = w[0].astype(np.float64)
        ax = [np.arange(n) / (n - 1) for n in (nx, ny, nz)]
        if dim == 2:
            e = sum(wd[i - 1, j - 1] * np.cos(i * np.pi * ax[0])[None, :] * np.cos(j * np.pi * ax[1])[:, None] / (1 + i * i + j * j)
                    for i in (1, 2) for j in (1, 2))
        else:
            e = sum(wd[i - 1, j - 1, k - 1] * np.cos(i * np.pi * ax[0])[None, None, :] * np.cos(j * np.pi * ax[1])[None, :, None]
                    * np.cos(k * np.pi * ax[2])[:, None, None] / (1 + i * i + j * j + k * k) for i in (1, 2) for j in (1, 2) for k in (1, 2))
        nu = np.exp(e)
        p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_KL_NODAL, kl_modes=2, kl_w=w, f_const=0.4)
        J = oracle.energy_grad(p, lin_profile(p.shape), want_r=False)
        tw = trapezoid_weights(dim, nx, ny, nz)
        assert J[1][0] == pytest.approx(0.5 * (tw * nu).sum(), rel=1e-13)            # diffusion part
        q = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, nu=nu[None].astype(np.float32), f_const=0.4)
        u = RNG.standard_normal(p.shape)
        a = oracle.energy_grad(p, u); b = oracle.energy_grad(q, u)
        assert a[0][0] == pytest.approx(b[0][0], rel=1e-6)
        assert np.abs(a[3] - b[3]).max() < 1e-6 * np.abs(b[3]).max()


def test_kl_gauss_mode_zero_weights_equals_unit_nodal():
    for dim, nx, ny, nz in GRIDS:
        p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2,
                    kl_w=np.zeros((1,) + (2,) * dim, np.float32), f_const=0.3)
        q = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, f_const=0.3); q.nu = const_nu(q, 1.0)
        u = RNG.standard_normal(p.shape)
        a = oracle.energy_grad(p, u); b = oracle.energy_grad(q, u)
        assert a[0][0] == pytest.approx(b[0][0], rel=1e-14) and np.allclose(a[3], b[3], atol=1e-13)


def test_kl_gauss_energy_of_linear_profile_converges_to_integral_of_nu():
    """u = 1 - x  =>  J = 1/2 * (Gauss quadrature of nu over the domain).  With the points in the right
    places the composite 2-point rule converges at 4th order to the true integral."""
    from scipy import integrate
    wv = 1.3
    w = np.zeros((1, 2, 2), np.float32); w[0, 0, 1] = wv                  # cos(pi x) cos(2 pi y) / 6
    wv = float(w[0, 0, 1])
    exact, _ = integrate.dblquad(lambda y, x: np.exp(wv * np.cos(np.pi * x) * np.cos(2 * np.pi * y) / 6.0),
                                 0, 1, 0, 1, epsabs=1e-13, epsrel=1e-13)
    errs = []
    for n in (5, 9, 17):
        p = Problem(dim=2, nx=n, ny=n + 2, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w)
        J = oracle.energy_grad(p, lin_profile(p.shape), want_r=False)[0][0]
        errs.append(abs(J - 0.5 * exact))
    # the integrand is even-periodic, so the composite rule converges faster than any power of h
    assert errs[0] < 1e-4 and errs[1] < 1e-9 and errs[2] < 1e-12, errs
    # 3D: tensor-product integrand  exp(w cos(pi x)cos(pi y)cos(pi z)/4), Gauss-Legendre reference
    w3 = np.zeros((1, 1, 1, 1), np.float32); w3[0, 0, 0, 0] = 1.1
    xg, wg = np.polynomial.legendre.leggauss(24)
    xg = 0.5 * (xg + 1); wg = 0.5 * wg
    c = np.cos(np.pi * xg)
    exact3 = np.einsum("i,j,k,ijk->", wg, wg, wg, np.exp(float(w3.ravel()[0]) * c[:, None, None] * c[None, :, None] * c[None, None, :] / 4.0))
    p = Problem(dim=3, nx=13, ny=11, nz=12, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=1, kl_w=w3)
    J = oracle.energy_grad(p, lin_profile(p.shape), want_r=False)[0][0]
    assert J == pytest.approx(0.5 * exact3, rel=2e-6)


def test_kl_gauss_points_written_out_on_one_and_two_elements():
    """u = 1 - x on a 1-element and a 3x2-element mesh: J = 1/2 sum_q W nu(x_q, y_q) with the Gauss points typed in."""
    g = 1.0 / np.sqrt(3.0)
    w = inputs.draw_weights(np.random.default_rng(8), 2, 2)[None]
    wd = w[0].astype(np.float64)

    def nu(x, y):
        return np.exp(sum(wd[i - 1, j - 1] * np.cos(i * np.pi * x) * np.cos(j * np.pi * y) / (1 + i * i + j * j)
                          for i in (1, 2) for j in (1, 2)))
    for nx, ny in ((2, 2), (4, 3)):
        hx, hy = 1.0 / (nx - 1), 1.0 / (ny - 1)
        ref = 0.0
        for ex in range(nx - 1):
            for ey in range(ny - 1):
                for sx in (-g, g):
                    for sy in (-g, g):
                        ref += 0.5 * (hx * hy / 4.0) * nu((ex + 0.5 + 0.5 * sx) * hx, (ey + 0.5 + 0.5 * sy) * hy)
        p = Problem(dim=2, nx=nx, ny=ny, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w)
        assert oracle.energy_grad(p, lin_profile(p.shape), want_r=False)[0][0] == pytest.approx(ref, rel=1e-14)
    # 3D, one element per axis except z: u = 1 - x, J = 1/2 sum_q W nu_q
    w3 = inputs.draw_weights(np.random.default_rng(9), 3, 2)[None]
    w3d = w3[0].astype(np.float64)
    nx, ny, nz = 2, 2, 3
    ref = 0.0
    for ez in range(nz - 1):
        for sx in (-g, g):
            for sy in (-g, g):
                for sz in (-g, g):
                    x, y, z = 0.5 + 0.5 * sx, 0.5 + 0.5 * sy, (ez + 0.5 + 0.5 * sz) / (nz - 1)
                    e = sum(w3d[i - 1, j - 1, k - 1] * np.cos(i * np.pi * x) * np.cos(j * np.pi * y) * np.cos(k * np.pi * z)
                            / (1 + i * i + j * j + k * k) for i in (1, 2) for j in (1, 2) for k in (1, 2))
                    ref += 0.5 * (1.0 / (nz - 1) / 8.0) * np.exp(e)
    p = Problem(dim=3, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w3)
    assert oracle.energy_grad(p, lin_profile(p.shape), want_r=False)[0][0] == pytest.approx(ref, rel=1e-14)


def _kl_nu_point(wd, *xyz):
    """The KL formula at one physical point, typed out (wd: float64 weights [m]^d)."""
    m = wd.shape[0]
    rng_ = range(1, m + 1)
    if len(xyz) == 2:
        x, y = xyz
        return np.exp(sum(wd[i - 1, j - 1] * np.cos(i * np.pi * x) * np.cos(j * np.pi * y) / (1 + i * i + j * j)
                          for i in rng_ for j in rng_))
    x, y, z = xyz
    return np.exp(sum(wd[i - 1, j - 1, k - 1] * np.cos(i * np.pi * x) * np.cos(j * np.pi * y) * np.cos(k * np.pi * z)
                      / (1 + i * i + j * j + k * k) for i in rng_ for j in rng_ for k in rng_))


def test_kl_gauss_energy_and_residual_of_fields_with_varying_gradient_written_out():
    """Which Gauss point's nu multiplies which gradient.  u = 2x + xy (2D) and u = x + xyz (3D) are Q1
    fields, so the interpolant is the field itself and grad u at a Gauss point is (2 + y, x) resp.
    (1 + yz, xz, xy) exactly, different at every point of an element; the energy is then the typed-out sum
    J = sum_e sum_q W 1/2 nu(x_q) |grad u(x_q)|^2 on non-square meshes with random weights.  The residual at
    one interior node is typed out the same way from the hat function's gradient."""
    g = 1.0 / np.sqrt(3.0)
    # ---- 2D, 3 x 4 nodes
    w = inputs.draw_weights(np.random.default_rng(21), 2, 2)[None]
    wd = w[0].astype(np.float64)
    nx, ny = 3, 4
    hx, hy = 1.0 / (nx - 1), 1.0 / (ny - 1)
    X = np.arange(nx) * hx; Y = np.arange(ny) * hy
    u = (2 * X[None, :] + X[None, :] * Y[:, None])[None]
    ref = 0.0
    # residual at the interior node (1, 2): its hat function is (1 - |x - X1|/hx)(1 - |y - Y2|/hy)
    ix, iy = 1, 2
    rref = 0.0
    for ex in range(nx - 1):
        for ey in range(ny - 1):
            for sx in (-g, g):
                for sy in (-g, g):
                    xq, yq = (ex + 0.5 + 0.5 * sx) * hx, (ey + 0.5 + 0.5 * sy) * hy
                    nuq = _kl_nu_point(wd, xq, yq)
                    gx, gy = 2.0 + yq, xq
                    W = hx * hy / 4.0
                    ref += W * 0.5 * nuq * (gx * gx + gy * gy)
                    if abs(xq - X[ix]) < hx and abs(yq - Y[iy]) < hy:
                        hxv, hyv = 1 - abs(xq - X[ix]) / hx, 1 - abs(yq - Y[iy]) / hy
                        dhx, dhy = -np.sign(xq - X[ix]) / hx, -np.sign(yq - Y[iy]) / hy
                        rref += W * nuq * (gx * dhx * hyv + gy * hxv * dhy)
    p = Problem(dim=2, nx=nx, ny=ny, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w, flags=NO_MASK)
    J, Jd, Jl, r = oracle.energy_grad(p, u)
    assert J[0] == pytest.approx(ref, rel=1e-13)
    assert r[0, iy, ix] == pytest.approx(rref, rel=1e-12)
    # ---- 3D, 2 x 3 x 2 nodes
    w3 = inputs.draw_weights(np.random.default_rng(22), 3, 2)[None]
    w3d = w3[0].astype(np.float64)
    nx, ny, nz = 2, 3, 2
    hx, hy, hz = 1.0 / (nx - 1), 1.0 / (ny - 1), 1.0 / (nz - 1)
    X = np.arange(nx) * hx; Y = np.arange(ny) * hy; Z = np.arange(nz) * hz
    u = (X[None, None, :] + X[None, None, :] * Y[None, :, None] * Z[:, None, None])[None]
    ref = 0.0
    ix, iy, iz = 1, 1, 0                                  # node on the x = 1 and z = 0 faces, interior in y
    rref = 0.0
    for ex in range(nx - 1):
        for ey in range(ny - 1):
            for ez in range(nz - 1):
                for sx in (-g, g):
                    for sy in (-g, g):
                        for sz in (-g, g):
                            xq, yq, zq = (ex + 0.5 + 0.5 * sx) * hx, (ey + 0.5 + 0.5 * sy) * hy, (ez + 0.5 + 0.5 * sz) * hz
                            nuq = _kl_nu_point(w3d, xq, yq, zq)
                            gr = (1.0 + yq * zq, xq * zq, xq * yq)
                            W = hx * hy * hz / 8.0
                            ref += W * 0.5 * nuq * (gr[0] ** 2 + gr[1] ** 2 + gr[2] ** 2)
                            d = (xq - X[ix], yq - Y[iy], zq - Z[iz])
                            hh = (hx, hy, hz)
                            if all(abs(d[a]) < hh[a] for a in range(3)):
                                v = [1 - abs(d[a]) / hh[a] for a in range(3)]
                                dv = [-np.sign(d[a]) / hh[a] for a in range(3)]
                                rref += W * nuq * (gr[0] * dv[0] * v[1] * v[2] + gr[1] * v[0] * dv[1] * v[2]
                                                   + gr[2] * v[0] * v[1] * dv[2])
    p = Problem(dim=3, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w3, flags=NO_MASK)
    J, Jd, Jl, r = oracle.energy_grad(p, u)
    assert J[0] == pytest.approx(ref, rel=1e-13)
    assert r[0, iz, iy, ix] == pytest.approx(rref, rel=1e-12)


def test_kl_gauss_converges_to_nodal_mode_under_refinement():
    """Both modes discretise the same continuous energy: their difference is O(h^2)."""
    w = inputs.draw_weights(np.random.default_rng(4), 2, 2)[None]
    diffs = []
    for n in (9, 17, 33):
        x = np.arange(n) / (n - 1)
        u = (1 - x)[None, None, :] + 0.2 * np.sin(2 * np.pi * x)[None, None, :] * np.cos(np.pi * x)[None, :, None]
        pk = Problem(dim=2, nx=n, ny=n, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w)
        pn = Problem(dim=2, nx=n, ny=n, batch=1, nu_mode=NU_NODAL, nu=oracle.kl_field(2, n, n, 1, 1, 2, w).astype(np.float32))
        diffs.append(abs(oracle.energy_grad(pk, u, want_r=False)[0][0] - oracle.energy_grad(pn, u, want_r=False)[0][0]))
    assert 3.0 < diffs[0] / diffs[1] < 5.0 and 3.0 < diffs[1] / diffs[2] < 5.0


# ---- interface semantics --------------------------------------------------------------------------
@pytest.mark.parametrize("dim,nx,ny,nz", GRIDS)
def test_apply_bc_mask_scale_and_sampled_residual(dim, nx, ny, nz):
    p = _problem(dim, nx, ny, nz, NU_KL_GAUSS, batch=3, f_const=0.5)
    p.flags = 0
    p.bc_x0, p.bc_x1 = 0.75, -0.25
    u = RNG.standard_normal(p.shape).astype(np.float32)
    ub = oracle.apply_bc(dim, nx, ny, nz, 3, p.bc_x0, p.bc_x1, 0, u.copy())
    assert np.all(ub[..., 0] == np.float32(0.75)) and np.all(ub[..., -1] == np.float32(-0.25))
    assert np.array_equal(ub[..., 1:-1], u[..., 1:-1])
    z = oracle.apply_bc(dim, nx, ny, nz, 3, 9, 9, 1, u.copy())
    assert np.all(z[..., 0] == 0) and np.all(z[..., -1] == 0) and np.array_equal(z[..., 1:-1], u[..., 1:-1])
    a = oracle.energy_grad(p, ub)
    p.flags = IMPOSE_BC_ON_LOAD
    b = oracle.energy_grad(p, u)                                  # imposition on load == apply_bc first
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[3], b[3])
    assert np.all(b[3][..., 0] == 0) and np.all(b[3][..., -1] == 0)
    gJ = np.array([2.0, -0.5, 0.0])
    c = oracle.energy_grad(p, u, gJ=gJ)
    assert np.allclose(c[3], b[3] * gJ.reshape((3,) + (1,) * dim), rtol=1e-15) and np.array_equal(c[0], b[0])
    idx = RNG.choice(u.size, size=60, replace=False)
    assert np.allclose(oracle.residual_at(p, u, idx, gJ=gJ), c[3].ravel()[idx], rtol=1e-13, atol=1e-15)


def test_threads_do_not_change_results():
    inp = inputs.make_inputs(0)
    p = Problem(dim=2, nx=64, ny=64, batch=8, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=inp.kl_w)
    n0 = oracle.num_threads()
    a = oracle.energy_grad(p, inp.u)
    oracle.set_num_threads(1)
    b = oracle.energy_grad(p, inp.u)
    oracle.set_num_threads(n0)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[3], b[3])


def test_input_recipe():
    a = inputs.make_inputs(0)
    b = inputs.make_inputs(0, samples=[3, 5])
    assert np.array_equal(a.u[[3, 5]], b.u) and np.array_equal(a.kl_w[[3, 5]], b.kl_w)
    assert np.all(a.u[..., 0] == 1.0) and np.all(a.u[..., -1] == 0.0)
    assert abs(a.kl_w).max() <= np.sqrt(3) and a.u.dtype == np.float32
    noise = a.u[..., 1:-1] - (1 - np.arange(64) / 63)[1:-1]
    assert 0.045 < noise.std() < 0.055
    s = inputs.sine_field(np.random.default_rng(0), 3, 12, 10, 8, 0.1, 32, 1.0, 0.0)
    # brute-force the same formula
    rng = np.random.default_rng(0)
    k = np.zeros((32, 3), dtype=np.int64)
    for i in range(32):
        while not k[i].any():
            k[i] = rng.integers(0, 5, size=3)
    phi = rng.uniform(0, 2 * np.pi, 32)
    X = np.arange(12) / 11; Y = np.arange(10) / 9; Z = np.arange(8) / 7
    ref = (1 - X)[None, None, :] + (0.1 / np.sqrt(32)) * sum(
        np.sin(2 * np.pi * (k[i, 0] * X[None, None, :] + k[i, 1] * Y[None, :, None] + k[i, 2] * Z[:, None, None]) + phi[i])
        for i in range(32))
    ref[..., 0] = 1; ref[..., -1] = 0
    assert np.allclose(s, ref.astype(np.float32), atol=1e-6)
