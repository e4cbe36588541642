"""The paper's split rule on the CUDA path ("Data Parallel Distributed Deep Learning": N_loc = ceil(N_s / p),
b_loc = floor(b_s / p), sequential draw; its result that the loss is the same for any number of workers p):
one mini-batch is cut into the shards p = 1, 2, 3, 4 workers would hold, the shards go through dn_energy_grad one
after another on one GPU, and the pieces must reproduce the unsharded call and the oracle's mean loss."""
import numpy as np
import pytest
import torch

import oracle
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs, sharding
from parity_util import dev

pytestmark = pytest.mark.gpu

N_SAMPLES = 12        # one mini-batch of 12 samples: divisible by 1, 2, 3, 4


def _run(inp, mode, sel):
    u = dev(inp.u[sel]); w = dev(inp.kl_w[sel])
    nb = len(sel)
    nu = None
    if mode == B.DN_NU_NODAL:
        nu = torch.empty(u.shape, device="cuda")
        B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, nb, inp.kl_modes, w, nu)
    p = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=nb, nu_mode=mode, nu=nu, kl_modes=inp.kl_modes,
                  kl_w=w, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    r = torch.full(u.shape, float("nan"), device="cuda"); J = torch.full((nb,), float("nan"), device="cuda")
    B.dn_energy_grad(p, u, None, J, r, B.new_workspace(p))
    torch.cuda.synchronize()
    return J.cpu().numpy(), r.cpu().numpy()


@pytest.mark.parametrize("dim,nx,ny,nz,m,mode", [
    (2, 256, 96, 1, 3, B.DN_NU_KL_GAUSS),          # tiled 2D kernel
    (2, 1024, 48, 1, 4, B.DN_NU_KL_GAUSS),         # strip 2D kernel
    (2, 1024, 48, 1, 4, B.DN_NU_NODAL),
    (3, 64, 24, 20, 2, B.DN_NU_KL_GAUSS),          # 3D
    (3, 128, 16, 12, 2, B.DN_NU_KL_NODAL),
    (2, 37, 29, 1, 2, B.DN_NU_KL_GAUSS),           # any-size kernel
])
def test_loss_and_gradient_do_not_depend_on_the_number_of_workers(dim, nx, ny, nz, m, mode):
    inp = inputs.random_inputs(dim, nx, ny, nz, N_SAMPLES, m, seed=77 + nx, f_const=0.5)
    J1, r1 = _run(inp, mode, list(range(N_SAMPLES)))
    omode = {B.DN_NU_KL_GAUSS: oracle.NU_KL_GAUSS, B.DN_NU_NODAL: oracle.NU_NODAL, B.DN_NU_KL_NODAL: oracle.NU_KL_NODAL}[mode]
    nu_o = None
    if mode == B.DN_NU_NODAL:                     # the field dn_kl_field wrote, read back, as in every nodal-mode parity test
        nu_t = torch.empty(inp.u.shape, device="cuda")
        B.dn_kl_field(dim, nx, ny, nz, N_SAMPLES, m, dev(inp.kl_w), nu_t)
        nu_o = nu_t.cpu().numpy()
    po = oracle.Problem(dim=dim, nx=nx, ny=ny, nz=nz, batch=N_SAMPLES, nu_mode=omode, nu=nu_o, kl_modes=m, kl_w=inp.kl_w,
                        f_const=0.5)
    Jo = oracle.energy_grad(po, inp.u, want_r=False)[0]
    rscale = np.abs(r1).max()
    for world in (1, 2, 3, 4):
        assert sharding.num_minibatches(N_SAMPLES, N_SAMPLES, world) == 1
        Js = np.empty(N_SAMPLES, np.float32); rs = np.empty_like(r1)
        for rank in range(world):
            sel = sharding.minibatch_indices(N_SAMPLES, N_SAMPLES, world, rank, 0)
            Js[sel], rs[sel] = _run(inp, mode, sel)
        # A sample's residual is a fixed sequence of operations on that sample alone: bit-identical however the batch
        # is cut (3D tiles may be cut differently for another batch size, which reorders two additions per seam node).
        if dim == 2:
            assert np.array_equal(rs, r1), f"p = {world}: residual differs from the unsharded call"
        else:
            assert np.abs(rs - r1).max() <= 1e-6 * rscale
        # The energy partials of a sample are summed over chunks whose height depends on the batch size: same value up
        # to the rounding of a double-precision sum
        assert np.all(np.abs(Js - J1) <= 1e-6 * np.abs(J1))
        # the averaged loss of Algorithm 1 (sum over ranks of local sums / global count) is the oracle's batch mean
        mean = sum(float(Js[sharding.minibatch_indices(N_SAMPLES, N_SAMPLES, world, rk, 0)].astype(np.float64).sum())
                   for rk in range(world)) / N_SAMPLES
        assert abs(mean - Jo.mean()) <= 1e-5 * abs(Jo.mean())
