"""Helpers of the GPU parity tests: the same numpy inputs go to the CPU oracle and to the CUDA library."""
import numpy as np
import torch

import oracle
from paper_2007_12792_b200 import binding as B

J_RTOL = 1e-5      # per sample |J - J*| <= J_RTOL |J*|
R_RTOL = 1e-5      # max |r - r*| <= R_RTOL max |r*|   (max over the whole batch tensor)


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def make_problems(inp, nu_mode, nu=None, f=None, flags=0, f_const=None, bc=None):
    """(oracle.Problem, binding.Problem) for the same inputs."""
    bc0, bc1 = bc if bc is not None else (inp.bc_x0, inp.bc_x1)
    fc = inp.f_const if f_const is None else f_const
    po = oracle.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=nu_mode, nu=nu,
                        kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=fc, f=f, bc_x0=bc0, bc_x1=bc1, flags=flags & 3)
    pg = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=nu_mode,
                   nu=dev(nu) if nu_mode == B.DN_NU_NODAL else None, kl_modes=inp.kl_modes,
                   kl_w=dev(inp.kl_w), f_const=fc, f=dev(f), bc_x0=bc0, bc_x1=bc1, flags=flags)
    return po, pg


def run_gpu(pg, u, gJ=None, want_J=True):
    ud = dev(u)
    r = torch.full(pg.shape, float("nan"), dtype=torch.float32, device="cuda")
    J = torch.full((pg.batch,), float("nan"), dtype=torch.float32, device="cuda") if want_J else None
    ws = B.new_workspace(pg)
    B.dn_energy_grad(pg, ud, dev(gJ), J, r, ws)
    torch.cuda.synchronize()
    return (J.cpu().numpy().astype(np.float64) if want_J else None), r.cpu().numpy().astype(np.float64)


def check(Jg, rg, Jo, ro, what=""):
    if Jg is not None:
        rel = np.abs(Jg - Jo) / np.abs(Jo)
        assert np.all(rel <= J_RTOL), f"{what}: J rel err {rel.max():.3e}  (J*={Jo}, J={Jg})"
    scale = np.abs(ro).max()
    err = np.abs(rg - ro).max()
    assert np.isfinite(rg).all(), f"{what}: non-finite residual"
    assert err <= R_RTOL * scale, f"{what}: r max err {err:.3e} vs scale {scale:.3e} ({err / scale:.3e})"
    return (0.0 if Jg is None else float((np.abs(Jg - Jo) / np.abs(Jo)).max())), float(err / max(scale, 1e-300))
