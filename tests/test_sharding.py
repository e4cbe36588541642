"""Sharding of the batch across ranks: the split rule on its own, and two gloo ranks on CPU that must
reproduce the single-process loss (the paper's "same problem for any number of workers")."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2007_12792_b200 import inputs, sharding


@pytest.mark.parametrize("n,b,p", [(4096, 1024, 4), (4096, 16, 1), (100, 8, 3), (37, 10, 2), (64, 64, 8), (7, 2, 2)])
def test_split_rule(n, b, p):
    n_loc, b_loc = sharding.local_counts(n, b, p)
    assert n_loc == int(np.ceil(n / p)) and b_loc == b // p
    nmb = sharding.num_minibatches(n, b, p)
    seen = []
    for mb in range(nmb):
        parts = [sharding.minibatch_indices(n, b, p, r, mb) for r in range(p)]
        assert len({len(x) for x in parts}) == 1                      # identical local sizes at any time
        union = [i for part in parts for i in part]
        single = sharding.minibatch_indices(p * n_loc, p * b_loc, 1, 0, mb)   # the adjusted single-process run
        assert union == single
        seen += union
    assert seen == list(range(p * n_loc))                             # every sample exactly once, in order


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, n_samples, batch, out):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    oracle.set_num_threads(1)
    losses = []
    for mb in range(sharding.num_minibatches(n_samples, batch, world)):
        idx = sharding.minibatch_indices(n_samples, batch, world, rank, mb)
        inp = inputs.make_inputs(0, samples=idx)
        p = oracle.Problem(dim=2, nx=inp.nx, ny=inp.ny, batch=inp.batch, nu_mode=oracle.NU_KL_GAUSS,
                           kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=inp.f_const)
        J = oracle.energy_grad(p, inp.u, want_r=False)[0]
        losses.append(sharding.mean_over_ranks(J.sum(), len(idx)))
    t = sharding.max_over_ranks([float(rank + 1), 5.0 - rank])
    if rank == 0:
        out.put((losses, t))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_process_loss():
    n_samples, batch, world = 12, 4, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_samples, batch, q)) for r in range(world)]
    for pr in procs:
        pr.start()
    losses, tmax = q.get(timeout=120)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    assert tmax == [2.0, 5.0]
    # single process, same adjusted sizes
    import oracle
    ref = []
    for mb in range(sharding.num_minibatches(n_samples, batch, 1)):
        idx = sharding.minibatch_indices(n_samples, batch, 1, 0, mb)
        inp = inputs.make_inputs(0, samples=idx)
        p = oracle.Problem(dim=2, nx=inp.nx, ny=inp.ny, batch=inp.batch, nu_mode=oracle.NU_KL_GAUSS,
                           kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=inp.f_const)
        ref.append(float(oracle.energy_grad(p, inp.u, want_r=False)[0].mean()))
    assert np.allclose(losses, ref, rtol=1e-13)
