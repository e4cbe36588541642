"""Plants plausible mistakes in a COPY of the oracle source (on the CPU) and checks that the pins notice each
one: a dropped term, a wrong sign, a wrong index, a misplaced Gauss point, a wrong weight, a transposed KL
index.  This is what "pinned" means for the oracle: the pin suite fails for every one of them."""
import ctypes as C
import os
import subprocess

import numpy as np
import pytest

import oracle
from oracle import Problem, NU_NODAL, NU_KL_GAUSS, NO_MASK

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "dn_oracle.cpp")

MUTATIONS = {
    "gauss_point_position": ("r.xi[0] = -1.0 / std::sqrt(3.0); r.xi[1] = 1.0 / std::sqrt(3.0);",
                             "r.xi[0] = -1.0 / 3.0; r.xi[1] = 1.0 / 3.0;"),
    "energy_half_dropped": ("Jdiff += W * 0.5 * nuq *", "Jdiff += W * nuq *"),
    "load_sign": ("- fq * N[a]);", "+ fq * N[a]);"),
    "y_gradient_dropped": ("gu[0] * dN[a][0] + gu[1] * dN[a][1] + gu[2] * dN[a][2]) - fq", "gu[0] * dN[a][0] + gu[2] * dN[a][2]) - fq"),
    "shape_derivative_scale": ("dfac[ax] = 0.5 * sgn * (2.0 / g.h[ax]);", "dfac[ax] = 0.5 * sgn * (1.0 / g.h[ax]);"),
    "quadrature_weight": ("double W = rule.wt[qx] * rule.wt[qy] * (g.h[0] / 2.0) * (g.h[1] / 2.0);",
                          "double W = rule.wt[qx] * rule.wt[qy] * (g.h[0] / 2.0) * (g.h[1]);"),
    "kl_denominator": ("(1.0 + (double)i * i + (double)j * j);", "(1.0 + (double)i * i + (double)j);"),
    "kl_axes_transposed_2d": ("std::cos(i * kPi * x) * std::cos(j * kPi * y) /\n                     (1.0",
                              "std::cos(j * kPi * x) * std::cos(i * kPi * y) /\n                     (1.0"),
    "gauss_point_in_wrong_element": ("const double x = (ex + 0.5 * (1.0 + ref[0])) * g.h[0];",
                                     "const double x = (ex + 1 + 0.5 * (1.0 + ref[0])) * g.h[0];"),
    "corner_index_swapped": ("const int ix = ex + (a & 1), iy = ey + ((a >> 1) & 1), iz = ez + ((a >> 2) & 1);\n        const long idx = node_index(g, ix, iy, iz);\n        uc[a]",
                             "const int ix = ex + ((a >> 1) & 1), iy = ey + (a & 1), iz = ez + ((a >> 2) & 1);\n        const long idx = node_index(g, ix, iy, iz);\n        uc[a]"),
    "mask_wrong_face": ("rb[node_index(g, g.nx - 1, iy, iz)] = 0.0;", "rb[node_index(g, g.nx - 2, iy, iz)] = 0.0;"),
    "kl_gauss_abscissae_swapped_between_axes": (
        "const double x = (ex + 0.5 * (1.0 + ref[0])) * g.h[0];\n                    const double y = (ey + 0.5 * (1.0 + ref[1])) * g.h[1];",
        "const double x = (ex + 0.5 * (1.0 + ref[1])) * g.h[0];\n                    const double y = (ey + 0.5 * (1.0 + ref[0])) * g.h[1];"),
    "kl_gauss_abscissae_shifted_cyclically_3d": (
        "const double y = (ey + 0.5 * (1.0 + ref[1])) * g.h[1];\n                    const double z = (g.dim == 3) ? (ez + 0.5 * (1.0 + ref[2])) * g.h[2] : 0.0;",
        "const double y = (ey + 0.5 * (1.0 + ref[g.dim == 3 ? 2 : 1])) * g.h[1];\n                    const double z = (g.dim == 3) ? (ez + 0.5 * (1.0 + ref[1])) * g.h[2] : 0.0;"),
    "nodal_nu_not_interpolated": ("nuq += N[a] * nuc[a];", "nuq += 0.125 * nuc[a] * (g.dim == 3 ? 1.0 : 2.0);"),
}


class _Mutant:
    """Minimal front end of a mutated oracle library (same C interface as the real one)."""

    def __init__(self, path):
        self.lib = C.CDLL(path)
        self.lib.orc_energy_grad.argtypes = [C.POINTER(oracle._Problem)] + [C.c_void_p] * 6
        self.lib.orc_kl_field.argtypes = [C.c_int] * 6 + [C.c_void_p, C.c_void_p]

    def energy_grad(self, p, u):
        s, uu, keep = oracle._marshal(p, u)
        J = np.empty(p.batch); Jd = np.empty(p.batch); Jl = np.empty(p.batch)
        r = np.empty(p.shape)
        assert self.lib.orc_energy_grad(C.byref(s), uu.ctypes.data, None, J.ctypes.data, Jd.ctypes.data, Jl.ctypes.data, r.ctypes.data) == 0
        return J, Jd, Jl, r

    def kl_field(self, nx, ny, w):
        out = np.empty((1, ny, nx))
        w = np.ascontiguousarray(w, dtype=np.float32)
        assert self.lib.orc_kl_field(2, nx, ny, 1, 1, w.shape[-1], w.ctypes.data, out.ctypes.data) == 0
        return out


def pins_hold(o) -> bool:
    """A condensed pin suite (closed forms only); returns False as soon as one pin is violated."""
    rng = np.random.default_rng(3)
    g = 1.0 / np.sqrt(3.0)
    for dim, nx, ny, nz in ((2, 7, 5, 1), (3, 4, 5, 3)):
        shape = (1, nz, ny, nx) if dim == 3 else (1, ny, nx)
        lin = np.broadcast_to(1.0 - np.arange(nx) / (nx - 1), shape).copy()
        # P1/P2: linear profile, constant nu
        p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, nu=np.full(shape, 2.5, np.float32), flags=NO_MASK)
        J, Jd, Jl, r = o.energy_grad(p, lin)
        if abs(J[0] - 1.25) > 1e-12 or np.abs(r[..., 1:-1]).max() > 1e-12:
            return False
        if abs(r[..., 0].sum() - 2.5) > 1e-11:
            return False
        # masked faces
        p.flags = 0
        u = rng.standard_normal(shape)
        rm = o.energy_grad(p, u)[3]
        if np.any(rm[..., 0] != 0) or np.any(rm[..., -1] != 0) or np.abs(rm[..., 1:-1]).max() == 0:
            return False
        if np.count_nonzero(rm[..., -2]) == 0:
            return False
        # P9: constant field, unit forcing
        p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, nu=np.full(shape, 1.0, np.float32), f_const=1.0, flags=NO_MASK)
        J, Jd, Jl, r = o.energy_grad(p, np.full(shape, 0.37))
        if abs(J[0] + 0.37) > 1e-12 or abs(r.sum() + 1.0) > 1e-12:
            return False
        # P10: nodal nu, linear profile: trapezoid energy
        nu = np.exp(0.3 * rng.standard_normal(shape)).astype(np.float32)
        w1 = lambda n: np.r_[0.5, np.ones(n - 2), 0.5] / (n - 1)
        tw = w1(ny)[:, None] * w1(nx)[None, :] if dim == 2 else w1(nz)[:, None, None] * w1(ny)[None, :, None] * w1(nx)[None, None, :]
        p = Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_NODAL, nu=nu, flags=NO_MASK)
        if abs(o.energy_grad(p, lin)[0][0] - 0.5 * (tw * nu[0].astype(np.float64)).sum()) > 1e-12:
            return False
        # P8: Euler identity, general u, anisotropic cells
        J, Jd, Jl, r = o.energy_grad(p, u)
        if abs(np.vdot(u, r) - 2 * Jd[0]) > 1e-10 * abs(Jd[0]):
            return False
    # one element, u = x y, bilinear nu: closed form from 1-D moments
    m0 = {0: 0.5, 1: 0.5}; m2 = {0: 1.0 / 12.0, 1: 0.25}
    nu1 = rng.uniform(0.5, 3.0, (1, 2, 2)).astype(np.float32)
    ref = 0.5 * sum(float(nu1[0, j, i]) * (m0[i] * m2[j] + m2[i] * m0[j]) for i in (0, 1) for j in (0, 1))
    p = Problem(dim=2, nx=2, ny=2, batch=1, nu_mode=NU_NODAL, nu=nu1)
    if abs(o.energy_grad(p, np.array([[[0.0, 0.0], [0.0, 1.0]]]))[0][0] - ref) > 1e-13:
        return False
    # KL field closed form with i != j
    w = np.zeros((1, 3, 3), np.float32); w[0, 0, 1] = 1.25
    x = np.arange(9) / 8; y = np.arange(6) / 5
    ref = np.exp(float(w[0, 0, 1]) * np.cos(np.pi * x)[None, :] * np.cos(2 * np.pi * y)[:, None] / 6.0)
    if not np.allclose(o.kl_field(9, 6, w)[0], ref, rtol=1e-12):
        return False
    # typed-out Gauss sum for KL at Gauss points, u = 1 - x on a 4 x 3 mesh
    wk = rng.uniform(-1.7, 1.7, (1, 2, 2)).astype(np.float32)
    wd = wk[0].astype(np.float64)
    nx, ny = 4, 3
    hx, hy = 1 / 3, 1 / 2
    ref = 0.0
    for ex in range(3):
        for ey in range(2):
            for sx in (-g, g):
                for sy in (-g, g):
                    X, Y = (ex + 0.5 + 0.5 * sx) * hx, (ey + 0.5 + 0.5 * sy) * hy
                    ref += 0.5 * (hx * hy / 4) * np.exp(sum(wd[i - 1, j - 1] * np.cos(i * np.pi * X) * np.cos(j * np.pi * Y) / (1 + i * i + j * j)
                                                            for i in (1, 2) for j in (1, 2)))
    p = Problem(dim=2, nx=nx, ny=ny, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=wk)
    lin = np.broadcast_to(1.0 - np.arange(nx) / (nx - 1), (1, ny, nx)).copy()
    if abs(o.energy_grad(p, lin)[0][0] - ref) > 1e-13:
        return False
    # typed-out Gauss sums for KL at Gauss points on Q1 fields whose gradient varies inside an element:
    # u = 2x + xy on 3 x 4 nodes, grad u = (2 + y, x);  u = x + xyz on 2 x 3 x 2 nodes, grad u = (1 + yz, xz, xy)
    nx, ny = 3, 4
    hx, hy = 1 / 2, 1 / 3
    X = np.arange(nx) * hx; Y = np.arange(ny) * hy
    ref = 0.0
    for ex in range(nx - 1):
        for ey in range(ny - 1):
            for sx in (-g, g):
                for sy in (-g, g):
                    xq, yq = (ex + 0.5 + 0.5 * sx) * hx, (ey + 0.5 + 0.5 * sy) * hy
                    nuq = np.exp(sum(wd[i - 1, j - 1] * np.cos(i * np.pi * xq) * np.cos(j * np.pi * yq) / (1 + i * i + j * j)
                                     for i in (1, 2) for j in (1, 2)))
                    ref += 0.5 * (hx * hy / 4) * nuq * ((2 + yq) ** 2 + xq ** 2)
    p = Problem(dim=2, nx=nx, ny=ny, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=wk)
    if abs(o.energy_grad(p, (2 * X[None, :] + X[None, :] * Y[:, None])[None])[0][0] - ref) > 1e-12 * ref:
        return False
    w3 = rng.uniform(-1.7, 1.7, (1, 2, 2, 2)).astype(np.float32)
    w3d = w3[0].astype(np.float64)
    nx, ny, nz = 2, 3, 2
    hx, hy, hz = 1.0, 0.5, 1.0
    X = np.arange(nx) * hx; Y = np.arange(ny) * hy; Z = np.arange(nz) * hz
    ref = 0.0
    for ey in range(ny - 1):
        for sx in (-g, g):
            for sy in (-g, g):
                for sz in (-g, g):
                    xq, yq, zq = (0.5 + 0.5 * sx) * hx, (ey + 0.5 + 0.5 * sy) * hy, (0.5 + 0.5 * sz) * hz
                    nuq = np.exp(sum(w3d[i - 1, j - 1, k - 1] * np.cos(i * np.pi * xq) * np.cos(j * np.pi * yq) * np.cos(k * np.pi * zq)
                                     / (1 + i * i + j * j + k * k) for i in (1, 2) for j in (1, 2) for k in (1, 2)))
                    ref += 0.5 * (hx * hy * hz / 8) * nuq * ((1 + yq * zq) ** 2 + (xq * zq) ** 2 + (xq * yq) ** 2)
    p = Problem(dim=3, nx=nx, ny=ny, nz=nz, batch=1, nu_mode=NU_KL_GAUSS, kl_modes=2, kl_w=w3)
    u3 = (X[None, None, :] + X[None, None, :] * Y[None, :, None] * Z[:, None, None])[None]
    if abs(o.energy_grad(p, u3)[0][0] - ref) > 1e-12 * ref:
        return False
    return True


class _Real:
    energy_grad = staticmethod(lambda p, u: oracle.energy_grad(p, u))
    kl_field = staticmethod(lambda nx, ny, w: oracle.kl_field(2, nx, ny, 1, 1, w.shape[-1], w))


def test_condensed_pins_hold_for_the_real_oracle():
    assert pins_hold(_Real)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation anchor for {name} not found exactly once"
    cpp = tmp_path / "mut.cpp"
    cpp.write_text(src.replace(old, new))
    so = tmp_path / "libmut.so"
    subprocess.run(["g++", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(so), str(cpp)], check=True)
    assert not pins_hold(_Mutant(str(so))), f"pins did not notice: {name}"
