"""Seeded synthetic inputs for the five workloads (numpy only).

This module draws inputs -- solution fields ``u`` and KL weights ``w`` -- and
nothing else: it contains none of the method's arithmetic (no diffusivity, no
energy, no residual) and imports neither the CUDA binding nor the CPU oracle, so
both sides can be fed the very same float32 arrays.

Recipe (one independent random stream per (workload, sample), so any subset of
samples can be produced on its own):

* ``w``      : ``[m]^dim`` values, uniform on ``(-sqrt(3), sqrt(3))`` (unit variance).
* ``noise`` u: ``(1 - x) + sigma * N(0,1)`` on every node with ``0 < ix < nx-1``;
               the faces ``ix = 0`` / ``ix = nx-1`` are set to ``bc_x0`` / ``bc_x1``.
* ``sines`` u: ``(1 - x) + (A / sqrt(M)) * sum_{s=1..M} sin(2 pi k_s . x + phi_s)``
               with integer wave vectors ``k_s`` drawn uniformly from ``{0..4}^dim``
               (the zero vector is redrawn) and phases uniform on ``[0, 2 pi)``;
               then the two faces are overwritten as above.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

BASE_SEED = 12792


@dataclass(frozen=True)
class Workload:
    index: int
    dim: int
    n: int            # nodes per axis
    batch: int
    kl_modes: int
    kind: str         # "noise" or "sines"
    sigma: float      # noise std, or sine amplitude A
    n_sines: int
    f_const: float
    bc_x0: float = 1.0
    bc_x1: float = 0.0

    @property
    def name(self) -> str:
        return f"cfg{self.index}_{self.dim}d_{self.n}^{self.dim}_b{self.batch}_m{self.kl_modes}"

    @property
    def grid(self):
        return (self.n, self.n, self.n if self.dim == 3 else 1)

    @property
    def nodes(self) -> int:
        return self.n ** self.dim

    @property
    def elements(self) -> int:
        return (self.n - 1) ** self.dim


WORKLOADS = (
    Workload(0, 2, 64, 8, 2, "noise", 0.05, 0, 0.0),
    Workload(1, 2, 256, 64, 4, "noise", 0.10, 0, 1.0),
    Workload(2, 2, 2048, 16, 6, "sines", 0.10, 16, 0.0),
    Workload(3, 3, 64, 32, 2, "noise", 0.05, 0, 0.0),
    Workload(4, 3, 256, 4, 3, "sines", 0.10, 32, 1.0),
)


def _rng(seed: int, sample: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([int(seed), int(sample)]))


def draw_weights(rng: np.random.Generator, dim: int, m: int) -> np.ndarray:
    r = np.sqrt(3.0)
    return rng.uniform(-r, r, size=(m,) * dim).astype(np.float32)


def _axis(n: int) -> np.ndarray:
    return np.arange(n, dtype=np.float64) / (n - 1)


def noise_field(rng, dim, nx, ny, nz, sigma, bc_x0, bc_x1) -> np.ndarray:
    shape = (nz, ny, nx) if dim == 3 else (ny, nx)
    u = np.broadcast_to(1.0 - _axis(nx), shape) + sigma * rng.standard_normal(shape)
    u[..., 0] = bc_x0
    u[..., -1] = bc_x1
    return u.astype(np.float32)


def sine_field(rng, dim, nx, ny, nz, amp, n_sines, bc_x0, bc_x1) -> np.ndarray:
    k = np.zeros((n_sines, dim), dtype=np.int64)
    for s in range(n_sines):
        while not k[s].any():
            k[s] = rng.integers(0, 5, size=dim)
    phi = rng.uniform(0.0, 2.0 * np.pi, size=n_sines)
    # sum_s sin(theta_x + theta_y (+ theta_z) + phi) as the imaginary part of a
    # sum of products of per-axis complex exponentials (one small matrix product).
    ex = np.exp(2j * np.pi * np.outer(k[:, 0], _axis(nx)))                     # [M][nx]
    ey = np.exp(2j * np.pi * np.outer(k[:, 1], _axis(ny)))                     # [M][ny]
    left = (ey * np.exp(1j * phi)[:, None]).T                                  # [ny][M]
    if dim == 3:
        ez = np.exp(2j * np.pi * np.outer(k[:, 2], _axis(nz)))                 # [M][nz]
        left = (ez.T[:, None, :] * left[None, :, :]).reshape(nz * ny, n_sines)
    a = np.concatenate([left.real, left.imag], axis=1)                         # [rows][2M]
    bmat = np.concatenate([ex.imag, ex.real], axis=0)                          # [2M][nx]
    s = (a @ bmat) * (amp / np.sqrt(n_sines))
    u = s.reshape((nz, ny, nx) if dim == 3 else (ny, nx)) + (1.0 - _axis(nx))
    u[..., 0] = bc_x0
    u[..., -1] = bc_x1
    return u.astype(np.float32)


@dataclass
class Inputs:
    workload: Optional[Workload]
    dim: int
    nx: int
    ny: int
    nz: int
    batch: int
    kl_modes: int
    kl_w: np.ndarray      # float32 [B][m]^dim
    u: np.ndarray         # float32 [B][nz][ny][nx] (3D) or [B][ny][nx] (2D)
    f_const: float
    bc_x0: float
    bc_x1: float
    seed: int
    samples: Sequence[int]


def make_inputs(index: int, samples: Optional[Sequence[int]] = None) -> Inputs:
    """Inputs of workload ``index``; ``samples`` selects a subset of its batch
    (default: all), each sample identical to what the full batch would hold."""
    wl = WORKLOADS[index]
    seed = BASE_SEED + 1000 * index
    if samples is None:
        samples = range(wl.batch)
    samples = list(samples)
    nx, ny, nz = wl.grid
    ws, us = [], []
    for b in samples:
        rng = _rng(seed, b)
        ws.append(draw_weights(rng, wl.dim, wl.kl_modes))
        if wl.kind == "noise":
            us.append(noise_field(rng, wl.dim, nx, ny, nz, wl.sigma, wl.bc_x0, wl.bc_x1))
        else:
            us.append(sine_field(rng, wl.dim, nx, ny, nz, wl.sigma, wl.n_sines, wl.bc_x0, wl.bc_x1))
    return Inputs(wl, wl.dim, nx, ny, nz, len(samples), wl.kl_modes, np.stack(ws), np.stack(us),
                  wl.f_const, wl.bc_x0, wl.bc_x1, seed, samples)


def random_inputs(dim: int, nx: int, ny: int, nz: int, batch: int, kl_modes: int, seed: int,
                  sigma: float = 0.1, f_const: float = 0.0, bc_x0: float = 1.0, bc_x1: float = 0.0) -> Inputs:
    """Noise-type inputs on an arbitrary grid (edge-case and odd-size tests)."""
    nzz = nz if dim == 3 else 1
    ws, us = [], []
    for b in range(batch):
        rng = _rng(seed, b)
        ws.append(draw_weights(rng, dim, kl_modes))
        us.append(noise_field(rng, dim, nx, ny, nzz, sigma, bc_x0, bc_x1))
    return Inputs(None, dim, nx, ny, nzz, batch, kl_modes, np.stack(ws), np.stack(us), f_const, bc_x0, bc_x1,
                  seed, list(range(batch)))


def random_positive_field(shape, seed: int, spread: float = 0.5) -> np.ndarray:
    """A positive float32 field (log-normal), used as a stand-in nodal coefficient in tests."""
    rng = np.random.default_rng(np.random.SeedSequence([int(seed), 7]))
    return np.exp(spread * rng.standard_normal(shape)).astype(np.float32)


def random_field(shape, seed: int, scale: float = 1.0) -> np.ndarray:
    rng = np.random.default_rng(np.random.SeedSequence([int(seed), 11]))
    return (scale * rng.standard_normal(shape)).astype(np.float32)


# ---- the paper's own workload: inviscid Burgers on (x, t) in [0,1] x [0, 0.2] -------------------------
@dataclass
class BurgersInputs:
    nx: int
    nt: int
    batch: int
    T: float
    lam: float
    c: np.ndarray         # float32 [B]: parameter of the initial-condition family
    u: np.ndarray         # float32 [B][nt][nx]: stand-in for a generator output
    seed: int


def burgers_inputs(nx: int, nt: int, batch: int, seed: int = BASE_SEED + 7000, noise: float = 0.01,
                   samples: Optional[Sequence[int]] = None) -> BurgersInputs:
    """Synthetic generator outputs for the Burgers loss: c ~ U(3, 6) (the paper's first example), the
    initial profile transported with speed 1/2, u = (1 - cos(2 pi c (x - t/2))) / 2, plus N(0, noise^2)."""
    if samples is None:
        samples = range(batch)
    samples = list(samples)
    x = _axis(nx)
    t = 0.2 * _axis(nt)
    cs, us = [], []
    for b in samples:
        rng = _rng(seed, b)
        c = np.float32(rng.uniform(3.0, 6.0))
        u = 0.5 * (1.0 - np.cos(2.0 * np.pi * float(c) * (x[None, :] - 0.5 * t[:, None]))) + noise * rng.standard_normal((nt, nx))
        cs.append(c)
        us.append(u.astype(np.float32))
    return BurgersInputs(nx, nt, len(samples), 0.2, 1.0, np.array(cs, dtype=np.float32), np.stack(us), seed)
