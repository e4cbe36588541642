"""Thin ctypes binding of ``libdn.so``: argument marshalling only.

The functions carry the names of the C entry points (``include/dn.h``).  Torch
tensors supply device memory and the current stream; every step of the path
runs in the library's CUDA kernels.  There is no CPU fallback: if the library
cannot be loaded, or a tensor is not a contiguous float32 CUDA tensor, the call
raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdn.so")

DN_OK = 0
DN_ERR_NULL, DN_ERR_DIM, DN_ERR_SIZE, DN_ERR_MODE, DN_ERR_WORKSPACE, DN_ERR_CUDA, DN_ERR_ALIAS = range(1, 8)
DN_NU_NODAL = 0
DN_NU_KL_GAUSS = 1
DN_NU_KL_NODAL = 2
DN_IMPOSE_BC_ON_LOAD = 1
DN_NO_MASK = 2
DN_FORCE_GENERIC = 4
DN_MAX_KL_MODES = 8

EXPORTS = ("dn_apply_bc_per_sample", "dn_workspace_bytes", "dn_host_staging_bytes", "dn_kl_field", "dn_energy", "dn_energy_grad",
           "dn_apply_bc", "dn_energy_grad_host", "dn_energy_grad_traced", "dn_energy_grad_static", "dn_launches_per_call", "dn_path_name", "dn_status_string",
           "dn_burgers_workspace_bytes", "dn_burgers_loss_grad", "dn_burgers_path_name",
           "dn_burgers_host_staging_bytes", "dn_burgers_loss_grad_host", "dn_cg_workspace_bytes", "dn_cg_solve")


class DnGrid(C.Structure):
    _fields_ = [("dim", C.c_int32), ("nx", C.c_int32), ("ny", C.c_int32), ("nz", C.c_int32)]


class DnProblem(C.Structure):
    _fields_ = [
        ("grid", DnGrid), ("batch", C.c_int32), ("nu_mode", C.c_int32), ("nu", C.c_void_p),
        ("kl_modes", C.c_int32), ("kl_w", C.c_void_p), ("f_const", C.c_float), ("f", C.c_void_p),
        ("bc_x0", C.c_float), ("bc_x1", C.c_float), ("flags", C.c_uint32),
        ("bc_x0_b", C.c_void_p), ("bc_x1_b", C.c_void_p),
    ]


class DnBurgers(C.Structure):
    _fields_ = [("nx", C.c_int32), ("nt", C.c_int32), ("batch", C.c_int32), ("T", C.c_float), ("lam", C.c_float),
                ("c", C.c_void_p), ("flags", C.c_uint32)]


class DnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} (status {int(status)})")


_lib = None


def lib():
    """Loads libdn.so (built by ``python -m paper_2007_12792_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2007_12792_b200.build`; "
                               "there is no fallback implementation")
        L = C.CDLL(LIB_PATH)
        PP = C.POINTER(DnProblem)
        PG = C.POINTER(DnGrid)
        L.dn_workspace_bytes.argtypes = [PP]; L.dn_workspace_bytes.restype = C.c_size_t
        L.dn_host_staging_bytes.argtypes = [PP]; L.dn_host_staging_bytes.restype = C.c_size_t
        L.dn_kl_field.argtypes = [PG, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.dn_energy.argtypes = [PP, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.dn_energy_grad.argtypes = [PP, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.dn_energy_grad_traced.argtypes = [PP, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                            C.c_void_p, C.c_void_p, C.c_void_p]
        L.dn_energy_grad_static.argtypes = [PP, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.dn_energy_grad_static.restype = C.c_int
        L.dn_apply_bc.argtypes = [PG, C.c_int32, C.c_float, C.c_float, C.c_int32, C.c_void_p, C.c_void_p]
        L.dn_apply_bc_per_sample.argtypes = [PG, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.dn_apply_bc_per_sample.restype = C.c_int
        L.dn_energy_grad_host.argtypes = [PP, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.dn_launches_per_call.argtypes = [PP]; L.dn_launches_per_call.restype = C.c_int32
        L.dn_path_name.argtypes = [PP]; L.dn_path_name.restype = C.c_char_p
        L.dn_status_string.argtypes = [C.c_int]; L.dn_status_string.restype = C.c_char_p
        L.dn_cg_workspace_bytes.argtypes = [PP]; L.dn_cg_workspace_bytes.restype = C.c_size_t
        L.dn_cg_solve.argtypes = [PP, C.c_void_p, C.c_int32, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                  C.c_void_p]
        L.dn_cg_solve.restype = C.c_int
        PB = C.POINTER(DnBurgers)
        L.dn_burgers_workspace_bytes.argtypes = [PB]; L.dn_burgers_workspace_bytes.restype = C.c_size_t
        L.dn_burgers_loss_grad.argtypes = [PB, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]
        L.dn_burgers_loss_grad.restype = C.c_int
        L.dn_burgers_host_staging_bytes.argtypes = [PB]; L.dn_burgers_host_staging_bytes.restype = C.c_size_t
        L.dn_burgers_loss_grad_host.argtypes = [PB, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                                C.c_size_t, C.c_void_p]
        L.dn_burgers_loss_grad_host.restype = C.c_int
        L.dn_burgers_path_name.argtypes = [PB, C.c_void_p, C.c_void_p]; L.dn_burgers_path_name.restype = C.c_char_p
        for f in ("dn_kl_field", "dn_energy", "dn_energy_grad", "dn_apply_bc", "dn_energy_grad_host", "dn_energy_grad_traced"):
            getattr(L, f).restype = C.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().dn_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor], name: str, device: str = "cuda") -> Optional[int]:
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name}: expected a torch.Tensor")
    if t.dtype != torch.float32 or not t.is_contiguous():
        raise ValueError(f"{name}: expected a contiguous float32 tensor")
    if device == "cuda" and not t.is_cuda:
        raise ValueError(f"{name}: expected a CUDA tensor (there is no CPU path)")
    if device == "cpu" and t.is_cuda:
        raise ValueError(f"{name}: expected a host tensor")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


@dataclass
class Problem:
    """Python mirror of ``dn_problem``; tensors must stay alive while work that uses them is in flight."""
    dim: int
    nx: int
    ny: int
    nz: int = 1
    batch: int = 1
    nu_mode: int = DN_NU_KL_GAUSS
    nu: Optional[torch.Tensor] = None
    kl_modes: int = 0
    kl_w: Optional[torch.Tensor] = None
    f_const: float = 0.0
    f: Optional[torch.Tensor] = None
    bc_x0: float = 1.0
    bc_x1: float = 0.0
    flags: int = 0
    bc_x0_b: Optional[torch.Tensor] = None      # [B] per-sample Dirichlet values; override the scalars
    bc_x1_b: Optional[torch.Tensor] = None

    @property
    def shape(self):
        return (self.batch, self.nz, self.ny, self.nx) if self.dim == 3 else (self.batch, self.ny, self.nx)

    def grid(self) -> DnGrid:
        return DnGrid(self.dim, self.nx, self.ny, self.nz if self.dim == 3 else 1)

    def c_struct(self, device: str = "cuda") -> DnProblem:
        p = DnProblem()
        p.grid = self.grid()
        p.batch, p.nu_mode, p.kl_modes = self.batch, self.nu_mode, self.kl_modes
        p.nu = _ptr(self.nu, "nu", device)
        p.kl_w = _ptr(self.kl_w, "kl_w", device)
        p.f = _ptr(self.f, "f", device)
        p.f_const, p.bc_x0, p.bc_x1, p.flags = self.f_const, self.bc_x0, self.bc_x1, self.flags
        p.bc_x0_b = _ptr(self.bc_x0_b, "bc_x0_b", device)
        p.bc_x1_b = _ptr(self.bc_x1_b, "bc_x1_b", device)
        return p


def dn_workspace_bytes(problem: Problem) -> int:
    return int(lib().dn_workspace_bytes(C.byref(problem.c_struct(device="any"))))


def dn_host_staging_bytes(problem: Problem) -> int:
    return int(lib().dn_host_staging_bytes(C.byref(problem.c_struct(device="any"))))


def dn_launches_per_call(problem: Problem) -> int:
    return int(lib().dn_launches_per_call(C.byref(problem.c_struct(device="any"))))


def dn_path_name(problem: Problem) -> str:
    return lib().dn_path_name(C.byref(problem.c_struct(device="any"))).decode()


def new_workspace(problem: Problem, device="cuda") -> torch.Tensor:
    """A device byte buffer of the size dn_workspace_bytes asks for (torch allocations are 256-B aligned or better)."""
    return torch.empty(max(dn_workspace_bytes(problem), 256), dtype=torch.uint8, device=device)


def new_host_staging(problem: Problem, device="cuda") -> torch.Tensor:
    return torch.empty(max(dn_host_staging_bytes(problem), 256), dtype=torch.uint8, device=device)


def _check(status: int, where: str):
    if status != DN_OK:
        raise DnError(status, where)


def dn_kl_field(dim: int, nx: int, ny: int, nz: int, batch: int, kl_modes: int, kl_w: torch.Tensor,
                nu_out: torch.Tensor, stream=None) -> torch.Tensor:
    g = DnGrid(dim, nx, ny, nz if dim == 3 else 1)
    _check(lib().dn_kl_field(C.byref(g), batch, kl_modes, _ptr(kl_w, "kl_w"), _ptr(nu_out, "nu_out"), _stream(stream)),
           "dn_kl_field")
    return nu_out


def dn_energy(problem: Problem, u: torch.Tensor, J: torch.Tensor, workspace: torch.Tensor, stream=None) -> torch.Tensor:
    p = problem.c_struct()
    _check(lib().dn_energy(C.byref(p), _ptr(u, "u"), _ptr(J, "J"), workspace.data_ptr(), workspace.numel(),
                           _stream(stream)), "dn_energy")
    return J


def dn_energy_grad(problem: Problem, u: torch.Tensor, gJ: Optional[torch.Tensor], J: Optional[torch.Tensor],
                   r: torch.Tensor, workspace: torch.Tensor, stream=None):
    p = problem.c_struct()
    _check(lib().dn_energy_grad(C.byref(p), _ptr(u, "u"), _ptr(gJ, "gJ"), _ptr(J, "J"), _ptr(r, "r"),
                                workspace.data_ptr(), workspace.numel(), _stream(stream)), "dn_energy_grad")
    return J, r


def dn_energy_grad_traced(problem: Problem, u: torch.Tensor, gJ: Optional[torch.Tensor], J: Optional[torch.Tensor],
                          r: torch.Tensor, workspace: torch.Tensor, event_before: Optional[torch.cuda.Event],
                          event_after: Optional[torch.cuda.Event], stream=None, _cstruct=None):
    """dn_energy_grad that records the two (already created, timing-enabled) torch CUDA events around
    the fused kernel.  ``_cstruct`` lets a tight loop reuse a marshalled ``dn_problem``."""
    p = _cstruct if _cstruct is not None else problem.c_struct()
    eb = None if event_before is None else event_before.cuda_event
    ea = None if event_after is None else event_after.cuda_event
    _check(lib().dn_energy_grad_traced(C.byref(p), _ptr(u, "u"), _ptr(gJ, "gJ"), _ptr(J, "J"), _ptr(r, "r"),
                                       workspace.data_ptr(), workspace.numel(), _stream(stream), eb, ea),
           "dn_energy_grad_traced")
    return J, r


def dn_energy_grad_static(problem: Problem, u: torch.Tensor, gJ: Optional[torch.Tensor], J: Optional[torch.Tensor],
                          r: torch.Tensor, stream=None):
    """dn_energy_grad for callers that may not allocate device memory (for instance code that runs under
    another framework's fixed memory plan): no workspace is passed, the library's built-in 1 MiB scratch
    array is used, and nothing is allocated here or in the library.  Problems that need more scratch raise
    DnError(DN_ERR_WORKSPACE).  Calls on one device share that array, so do not overlap them on the GPU."""
    p = problem.c_struct()
    _check(lib().dn_energy_grad_static(C.byref(p), _ptr(u, "u"), _ptr(gJ, "gJ"), _ptr(J, "J"), _ptr(r, "r"),
                                       _stream(stream)), "dn_energy_grad_static")
    return J, r


def dn_apply_bc(dim: int, nx: int, ny: int, nz: int, batch: int, bc_x0: float, bc_x1: float, mode: int,
                field: torch.Tensor, stream=None) -> torch.Tensor:
    g = DnGrid(dim, nx, ny, nz if dim == 3 else 1)
    _check(lib().dn_apply_bc(C.byref(g), batch, bc_x0, bc_x1, mode, _ptr(field, "field"), _stream(stream)), "dn_apply_bc")
    return field


def dn_apply_bc_per_sample(dim: int, nx: int, ny: int, nz: int, batch: int, bc_x0_b: torch.Tensor, bc_x1_b: torch.Tensor,
                           field: torch.Tensor, stream=None) -> torch.Tensor:
    g = DnGrid(dim, nx, ny, nz if dim == 3 else 1)
    _check(lib().dn_apply_bc_per_sample(C.byref(g), batch, _ptr(bc_x0_b, "bc_x0_b"), _ptr(bc_x1_b, "bc_x1_b"),
                                        _ptr(field, "field"), _stream(stream)), "dn_apply_bc_per_sample")
    return field


def dn_energy_grad_host(problem: Problem, u_host: torch.Tensor, gJ_host: Optional[torch.Tensor],
                        J_host: Optional[torch.Tensor], r_host: torch.Tensor, staging: torch.Tensor, stream=None):
    """Host-buffer variant: ``problem.nu / kl_w / f`` and all tensors here are HOST tensors (pinned for speed);
    ``staging`` is a device byte buffer of dn_host_staging_bytes(problem).  Returns after the results are on the host."""
    p = problem.c_struct(device="cpu")
    _check(lib().dn_energy_grad_host(C.byref(p), _ptr(u_host, "u_host", "cpu"), _ptr(gJ_host, "gJ_host", "cpu"),
                                     _ptr(J_host, "J_host", "cpu"), _ptr(r_host, "r_host", "cpu"),
                                     staging.data_ptr(), staging.numel(), _stream(stream)), "dn_energy_grad_host")
    return J_host, r_host


@dataclass
class Burgers:
    """Python mirror of ``dn_burgers`` (the paper's Burgers finite-difference loss)."""
    nx: int
    nt: int
    batch: int
    c: Optional[torch.Tensor] = None      # [B] float32 wave numbers of the initial-condition family
    T: float = 0.2
    lam: float = 1.0
    flags: int = 0

    @property
    def shape(self):
        return (self.batch, self.nt, self.nx)

    def c_struct(self, device: str = "cuda") -> DnBurgers:
        p = DnBurgers()
        p.nx, p.nt, p.batch, p.T, p.lam, p.flags = self.nx, self.nt, self.batch, self.T, self.lam, self.flags
        p.c = _ptr(self.c, "c", device)
        return p


def dn_burgers_workspace_bytes(problem: Burgers) -> int:
    return int(lib().dn_burgers_workspace_bytes(C.byref(problem.c_struct(device="any"))))


def dn_burgers_path_name(problem: Burgers, u: Optional[torch.Tensor], g: Optional[torch.Tensor]) -> str:
    return lib().dn_burgers_path_name(C.byref(problem.c_struct(device="any")), _ptr(u, "u", "any"), _ptr(g, "g", "any")).decode()


def new_burgers_workspace(problem: Burgers, device="cuda") -> torch.Tensor:
    return torch.empty(max(dn_burgers_workspace_bytes(problem), 256), dtype=torch.uint8, device=device)


def dn_burgers_loss_grad(problem: Burgers, u: torch.Tensor, gL: Optional[torch.Tensor], L: Optional[torch.Tensor],
                         parts: Optional[torch.Tensor], g: Optional[torch.Tensor], workspace: torch.Tensor, stream=None,
                         event_before: Optional[torch.cuda.Event] = None, event_after: Optional[torch.cuda.Event] = None,
                         _cstruct=None):
    """L[b] = L_p + lam L_b, parts[b] = (L_p, L_b) and g = dL/du (times gL[b]) of the Burgers loss; any of L, parts,
    g may be None.  The two optional (created, timing-enabled) events are recorded around the main kernel."""
    p = _cstruct if _cstruct is not None else problem.c_struct()
    eb = None if event_before is None else event_before.cuda_event
    ea = None if event_after is None else event_after.cuda_event
    _check(lib().dn_burgers_loss_grad(C.byref(p), _ptr(u, "u"), _ptr(gL, "gL"), _ptr(L, "L"), _ptr(parts, "parts"),
                                      _ptr(g, "g"), workspace.data_ptr(), workspace.numel(), _stream(stream), eb, ea),
           "dn_burgers_loss_grad")
    return L, parts, g


def dn_burgers_host_staging_bytes(problem: Burgers) -> int:
    return int(lib().dn_burgers_host_staging_bytes(C.byref(problem.c_struct(device="any"))))


def new_burgers_host_staging(problem: Burgers, device="cuda") -> torch.Tensor:
    return torch.empty(max(dn_burgers_host_staging_bytes(problem), 256), dtype=torch.uint8, device=device)


def dn_burgers_loss_grad_host(problem: Burgers, u_host: torch.Tensor, gL_host: Optional[torch.Tensor],
                              L_host: Optional[torch.Tensor], parts_host: Optional[torch.Tensor], g_host: torch.Tensor,
                              staging: torch.Tensor, stream=None):
    """Host-buffer variant: ``problem.c`` and all tensors are HOST tensors (pinned for speed); ``staging`` is a device
    byte buffer of dn_burgers_host_staging_bytes(problem).  Returns after the results are on the host."""
    p = problem.c_struct(device="cpu")
    _check(lib().dn_burgers_loss_grad_host(C.byref(p), _ptr(u_host, "u_host", "cpu"), _ptr(gL_host, "gL_host", "cpu"),
                                           _ptr(L_host, "L_host", "cpu"), _ptr(parts_host, "parts_host", "cpu"),
                                           _ptr(g_host, "g_host", "cpu"), staging.data_ptr(), staging.numel(),
                                           _stream(stream)), "dn_burgers_loss_grad_host")
    return L_host, parts_host, g_host


def dn_cg_workspace_bytes(problem: Problem) -> int:
    return int(lib().dn_cg_workspace_bytes(C.byref(problem.c_struct(device="any"))))


def new_cg_workspace(problem: Problem, device="cuda") -> torch.Tensor:
    return torch.empty(max(dn_cg_workspace_bytes(problem), 256), dtype=torch.uint8, device=device)


def dn_cg_solve(problem: Problem, u: torch.Tensor, max_iters: int, rtol: float, relres: Optional[torch.Tensor],
                iters: Optional[torch.Tensor], workspace: torch.Tensor, stream=None):
    """Solves K(nu) u = F in place (matrix-free Jacobi-preconditioned CG on the fused kernel); relres: [B] float32,
    iters: [B] int32 device tensors or None.  Enqueues exactly max_iters iterations."""
    if iters is not None and (iters.dtype != torch.int32 or not iters.is_cuda or not iters.is_contiguous()):
        raise ValueError("iters: expected a contiguous int32 CUDA tensor")
    p = problem.c_struct()
    _check(lib().dn_cg_solve(C.byref(p), _ptr(u, "u"), int(max_iters), float(rtol), _ptr(relres, "relres"),
                             None if iters is None else iters.data_ptr(), workspace.data_ptr(), workspace.numel(),
                             _stream(stream)), "dn_cg_solve")
    return u
