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


GUARD = 4096          # sentinel bytes before and after every output buffer and the workspace
_SENTINEL = 0xA5


def guarded(nbytes, dtype=torch.uint8):
    """(whole, view): a device byte buffer filled with a sentinel, and the nbytes in its middle (GUARD bytes of
    sentinel on either side; GUARD is a multiple of 256, so the view keeps the allocation's alignment)."""
    whole = torch.full((nbytes + 2 * GUARD,), _SENTINEL, dtype=torch.uint8, device="cuda")
    return whole, whole[GUARD:GUARD + nbytes]


def guards_intact(whole, nbytes):
    """Nothing wrote outside the middle nbytes (the stand-in for a memory checker: a kernel that stores one
    element before or after r, J or its workspace changes a sentinel byte)."""
    return bool((whole[:GUARD] == _SENTINEL).all()) and bool((whole[GUARD + nbytes:] == _SENTINEL).all())


def run_gpu(pg, u, gJ=None, want_J=True):
    ud = dev(u)
    n = int(np.prod(pg.shape))
    r_whole, r_bytes = guarded(4 * n)
    r = r_bytes.view(torch.float32).view(pg.shape)
    r.fill_(float("nan"))
    J_whole, J_bytes = guarded(4 * pg.batch)
    J = J_bytes.view(torch.float32)
    J.fill_(float("nan"))
    ws_n = max(B.dn_workspace_bytes(pg), 256)
    ws_whole, ws = guarded(ws_n)
    B.dn_energy_grad(pg, ud, dev(gJ), J if want_J else None, r, ws)
    torch.cuda.synchronize()
    assert guards_intact(r_whole, 4 * n), "bytes outside r were written"
    assert guards_intact(J_whole, 4 * pg.batch), "bytes outside J were written"
    assert guards_intact(ws_whole, ws_n), "bytes outside the workspace were written"
    if not want_J:
        assert bool(torch.isnan(J).all()), "J was written although it was not asked for"
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
