"""One population spread over several GPUs by antithetic pairs (paper Section 2, "Device
Parallelism").  Rank r owns pairs [r*H/W, (r+1)*H/W): it samples and evaluates only those (the
noise of a pair comes from counters, so none is exchanged) and the generation needs exactly two
small exchanges: an all-gather of P fitness floats and an all-reduce of the D-long gradient sums.
Every rank then applies the same update and ends with the same centre.

The exchange functions take any torch.distributed process group (NCCL on GPUs; the CPU tests run
them over gloo).
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def shard_of(n_pairs: int, rank: int, world: int) -> Tuple[int, int]:
    """(first pair, number of pairs) of `rank`; the pairs must divide evenly (all-gather of equal parts)."""
    if n_pairs % world != 0:
        raise ValueError(f"{n_pairs} antithetic pairs do not divide over {world} ranks")
    per = n_pairs // world
    return rank * per, per


def gather_fitness(fit_local: torch.Tensor, world: int, group=None) -> torch.Tensor:
    """Global fitness vector in member order from the ranks' contiguous shards."""
    if world == 1:
        return fit_local
    out = torch.empty(fit_local.numel() * world, dtype=fit_local.dtype, device=fit_local.device)
    dist.all_gather_into_tensor(out, fit_local.contiguous(), group=group)
    return out


def reduce_sums(grad_sum: torch.Tensor, sigma_sum: Optional[torch.Tensor], world: int, group=None) -> None:
    """Sums the per-shard gradient sums over the ranks, in place (every rank gets the same bits)."""
    if world == 1:
        return
    dist.all_reduce(grad_sum, op=dist.ReduceOp.SUM, group=group)
    if sigma_sum is not None:
        dist.all_reduce(sigma_sum, op=dist.ReduceOp.SUM, group=group)


def generation(solver, world: int, group=None, fitness_local: Optional[torch.Tensor] = None) -> torch.Tensor:
    """ask -> rollout -> exchange -> update on one rank's sharded solver; returns the global fitness."""
    solver.ask()
    fit_local = solver.rollout() if fitness_local is None else fitness_local
    fit_all = gather_fitness(fit_local, world, group)
    solver.tell_begin(fit_all)
    grad_sum, sigma_sum = solver.reduce_buffers()
    reduce_sums(grad_sum, sigma_sum, world, group)
    solver.tell_end()
    return fit_all
