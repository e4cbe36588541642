"""TEST INFRASTRUCTURE -- not part of the product.

ctypes front end of the plain fp64 CPU oracle (``dn_oracle.cpp``).  Only the
tests, the smoke check and the CPU-baseline leg of the benchmark may import it;
the CUDA library and its Python binding never do.

All arrays are numpy, C-ordered ``[B][nz][ny][nx]`` (x fastest).  Inputs that
the GPU path also receives (``u``, ``nu``, ``kl_w``, ``f``) are float32 and are
promoted to double inside the oracle; results are float64.

Parity pins live in ``tests/test_oracle_pins.py``; every function is pinned (the
KL-at-Gauss mode by Gauss sums typed out point by point on Q1 fields whose
gradient varies inside an element).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dn_oracle.cpp")
_LIB = os.path.join(_HERE, "libdn_oracle.so")

NU_NODAL = 0
NU_KL_GAUSS = 1
NU_KL_NODAL = 2
IMPOSE_BC_ON_LOAD = 1
NO_MASK = 2


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (fp64, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-ffp-contract=off", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


class _Problem(C.Structure):
    _fields_ = [
        ("dim", C.c_int32), ("nx", C.c_int32), ("ny", C.c_int32), ("nz", C.c_int32), ("batch", C.c_int32),
        ("nu_mode", C.c_int32), ("kl_modes", C.c_int32), ("nquad", C.c_int32),
        ("flags", C.c_uint32), ("u_f64", C.c_int32),
        ("f_const", C.c_double), ("bc_x0", C.c_double), ("bc_x1", C.c_double),
        ("nu", C.c_void_p), ("kl_w", C.c_void_p), ("f", C.c_void_p),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        lib = C.CDLL(_LIB)
        lib.orc_num_threads.restype = C.c_int
        lib.orc_set_num_threads.argtypes = [C.c_int]
        lib.orc_kl_field.argtypes = [C.c_int] * 6 + [C.c_void_p, C.c_void_p]
        lib.orc_energy_grad.argtypes = [C.POINTER(_Problem)] + [C.c_void_p] * 6
        lib.orc_residual_at.argtypes = [C.POINTER(_Problem), C.c_void_p, C.c_void_p, C.c_long, C.c_void_p, C.c_void_p]
        lib.orc_apply_bc.argtypes = [C.c_int] * 5 + [C.c_double, C.c_double, C.c_int, C.c_void_p]
        lib.orc_assemble.argtypes = [C.POINTER(_Problem), C.c_int, C.c_void_p, C.c_void_p]
        lib.orc_solve_dirichlet.argtypes = [C.c_int] * 4 + [C.c_void_p, C.c_void_p, C.c_double, C.c_double, C.c_void_p]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def set_num_threads(n: int) -> None:
    _load().orc_set_num_threads(int(n))


@dataclass
class Problem:
    """Arguments of one oracle call; mirrors the statement of the problem:
    grid size, batch, KL coefficients (or a nodal nu), boundary values, forcing."""
    dim: int
    nx: int
    ny: int
    nz: int = 1
    batch: int = 1
    nu_mode: int = NU_NODAL
    nu: Optional[np.ndarray] = None        # float32 [B][nz][ny][nx]
    kl_modes: int = 0
    kl_w: Optional[np.ndarray] = None      # float32 [B][m]^dim
    f_const: float = 0.0
    f: Optional[np.ndarray] = None         # float32 nodal forcing or None
    bc_x0: float = 1.0
    bc_x1: float = 0.0
    flags: int = 0
    nquad: int = 2

    @property
    def shape(self):
        return (self.batch, self.nz, self.ny, self.nx) if self.dim == 3 else (self.batch, self.ny, self.nx)

    @property
    def nodes(self) -> int:
        return self.nx * self.ny * (self.nz if self.dim == 3 else 1)


def _f32(a, n, name):
    a = np.ascontiguousarray(a, dtype=np.float32)
    if a.size != n:
        raise ValueError(f"{name}: expected {n} values, got {a.size}")
    return a


def _marshal(p: Problem, u):
    keep = []
    s = _Problem()
    s.dim, s.nx, s.ny, s.nz, s.batch = p.dim, p.nx, p.ny, (p.nz if p.dim == 3 else 1), p.batch
    s.nu_mode, s.kl_modes, s.nquad, s.flags = p.nu_mode, p.kl_modes, p.nquad, p.flags
    s.f_const, s.bc_x0, s.bc_x1 = float(p.f_const), float(p.bc_x0), float(p.bc_x1)
    ntot = p.batch * p.nodes
    if p.nu_mode == NU_NODAL:
        nu = _f32(p.nu, ntot, "nu"); keep.append(nu); s.nu = nu.ctypes.data
    else:
        w = _f32(p.kl_w, p.batch * p.kl_modes ** p.dim, "kl_w"); keep.append(w); s.kl_w = w.ctypes.data
    if p.f is not None:
        f = _f32(p.f, ntot, "f"); keep.append(f); s.f = f.ctypes.data
    uu = None
    if u is not None:
        u = np.asarray(u)
        if u.dtype == np.float64:
            uu = np.ascontiguousarray(u); s.u_f64 = 1
        else:
            uu = np.ascontiguousarray(u, dtype=np.float32); s.u_f64 = 0
        if uu.size != ntot:
            raise ValueError(f"u: expected {ntot} values, got {uu.size}")
        keep.append(uu)
    return s, uu, keep


def kl_field(dim, nx, ny, nz, batch, kl_modes, kl_w) -> np.ndarray:
    """nu at the grid nodes from the KL formula (float64)."""
    nzz = nz if dim == 3 else 1
    w = _f32(kl_w, batch * kl_modes ** dim, "kl_w")
    out = np.empty((batch, nzz, ny, nx) if dim == 3 else (batch, ny, nx), dtype=np.float64)
    rc = _load().orc_kl_field(dim, nx, ny, nzz, batch, kl_modes, w.ctypes.data, out.ctypes.data)
    if rc:
        raise ValueError("orc_kl_field: invalid arguments")
    return out


def energy_grad(p: Problem, u, gJ=None, want_r: bool = True):
    """Returns (J[B], Jdiff[B], Jload[B], r or None), all float64.  J = Jdiff - Jload."""
    s, uu, keep = _marshal(p, u)
    J = np.empty(p.batch); Jd = np.empty(p.batch); Jl = np.empty(p.batch)
    r = np.empty(p.shape, dtype=np.float64) if want_r else None
    g = None if gJ is None else np.ascontiguousarray(gJ, dtype=np.float64)
    rc = _load().orc_energy_grad(C.byref(s), uu.ctypes.data, None if g is None else g.ctypes.data,
                                 J.ctypes.data, Jd.ctypes.data, Jl.ctypes.data,
                                 None if r is None else r.ctypes.data)
    if rc:
        raise ValueError("orc_energy_grad: invalid arguments")
    return J, Jd, Jl, r


def residual_at(p: Problem, u, flat_idx, gJ=None) -> np.ndarray:
    """Residual at the nodes whose flat indices into [B][nz][ny][nx] are given."""
    s, uu, keep = _marshal(p, u)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    out = np.empty(idx.size, dtype=np.float64)
    g = None if gJ is None else np.ascontiguousarray(gJ, dtype=np.float64)
    rc = _load().orc_residual_at(C.byref(s), uu.ctypes.data, None if g is None else g.ctypes.data,
                                 idx.size, idx.ctypes.data, out.ctypes.data)
    if rc:
        raise ValueError("orc_residual_at: invalid arguments")
    return out


def apply_bc(dim, nx, ny, nz, batch, bc_x0, bc_x1, mode, field: np.ndarray) -> np.ndarray:
    """Overwrites the two x faces of a float32 field in place and returns it."""
    if field.dtype != np.float32 or not field.flags.c_contiguous:
        raise ValueError("field must be contiguous float32")
    nzz = nz if dim == 3 else 1
    rc = _load().orc_apply_bc(dim, nx, ny, nzz, batch, float(bc_x0), float(bc_x1), int(mode), field.ctypes.data)
    if rc:
        raise ValueError("orc_apply_bc: invalid arguments")
    return field


def assemble(p: Problem, b: int = 0):
    """Dense K [n][n] and F [n] of sample b (tiny grids)."""
    s, _, keep = _marshal(p, None)
    n = p.nodes
    K = np.empty((n, n)); F = np.empty(n)
    rc = _load().orc_assemble(C.byref(s), b, K.ctypes.data, F.ctypes.data)
    if rc:
        raise ValueError("orc_assemble: invalid arguments")
    return K, F


def solve_dirichlet(p: Problem, K, F) -> np.ndarray:
    """Discrete solution with the two x faces fixed (Gaussian elimination), shape of one sample."""
    K = np.ascontiguousarray(K, dtype=np.float64); F = np.ascontiguousarray(F, dtype=np.float64)
    u = np.empty(p.nodes)
    nzz = p.nz if p.dim == 3 else 1
    rc = _load().orc_solve_dirichlet(p.dim, p.nx, p.ny, nzz, K.ctypes.data, F.ctypes.data,
                                     float(p.bc_x0), float(p.bc_x1), u.ctypes.data)
    if rc:
        raise ValueError("orc_solve_dirichlet failed")
    return u.reshape(p.shape[1:])
