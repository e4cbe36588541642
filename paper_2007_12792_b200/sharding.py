"""Batch sharding across ranks: samples are independent, so the path shards by whole samples with
no collective on the data path; only the scalar loss is averaged.

Follows the paper's data-parallel rule ("Data Parallel Distributed Deep Learning", the two
equations for the local sample count and batch size, and Algorithm 1): the sample count N_s and
batch size b_s are adjusted so that every rank draws N_loc = ceil(N_s / p) samples in
mini-batches of b_loc = floor(b_s / p), sequentially from the global pool, such that the union of
the local mini-batches equals the mini-batch of a single-process run with the adjusted sizes.
"""
from __future__ import annotations

from typing import List, Tuple


def local_counts(n_samples: int, batch: int, world: int) -> Tuple[int, int]:
    """(N_loc, b_loc) = (ceil(N_s / p), floor(b_s / p))."""
    if world < 1 or n_samples < 1 or batch < world:
        raise ValueError("need world >= 1, n_samples >= 1 and batch >= world")
    return -(-n_samples // world), batch // world


def num_minibatches(n_samples: int, batch: int, world: int) -> int:
    n_loc, b_loc = local_counts(n_samples, batch, world)
    return -(-n_loc // b_loc)


def minibatch_indices(n_samples: int, batch: int, world: int, rank: int, mb: int) -> List[int]:
    """Global sample indices that `rank` processes in mini-batch `mb`.

    The global mini-batch `mb` of the adjusted problem (p N_loc samples, batches of p b_loc) is the
    contiguous range a single process would draw; it is cut into `world` equal contiguous pieces.
    The last, shorter mini-batch has p (N_loc mod b_loc) samples, again divisible by p, so all ranks
    always hold the same number of samples."""
    n_loc, b_loc = local_counts(n_samples, batch, world)
    if not (0 <= rank < world) or not (0 <= mb < num_minibatches(n_samples, batch, world)):
        raise ValueError("rank or mini-batch out of range")
    start = mb * b_loc * world
    size = min(b_loc, n_loc - mb * b_loc)          # local size of this mini-batch
    lo = start + rank * size
    return list(range(lo, lo + size))


def mean_over_ranks(local_sum, local_count, group=None):
    """Average of per-sample losses over the global mini-batch (Algorithm 1, averaged loss): one
    all-reduce of two scalars.  Works on any torch.distributed backend; returns a Python float."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(local_sum), float(local_count)], dtype=torch.float64)
    if dist.is_available() and dist.is_initialized():
        if dist.get_backend(group) == "nccl":
            t = t.cuda()
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t[0] / t[1])


def max_over_ranks(values, group=None):
    """Element-wise maximum over ranks of a short list of floats (device timings)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64)
    if dist.is_available() and dist.is_initialized():
        if dist.get_backend(group) == "nccl":
            t = t.cuda()
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return [float(x) for x in t.cpu()]
