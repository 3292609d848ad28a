"""Host logic of running the step as independent replicas, one process per GPU.

The draft-and-verify step has no exchange between sequences (the method is described for one
sequence at a time), so N GPUs run N replicas: every rank drafts its own sequences, no collective
touches the data path, and the only communication is the timing protocol below (a barrier around
the timed region and the maximum of the ranks' times).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import synth


def rank_workload(w: synth.Workload, rank: int) -> synth.Workload:
    """The workload of one rank: same shapes, its own seed, so that every rank drafts other sequences."""
    return synth.scaled(w, seed=w.seed + 17 * rank)


def max_over_ranks(x: float, device) -> float:
    """Maximum of `x` over all ranks (x itself when no process group is up)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_steps_per_s(world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank completes one step per `ms_per_step` (weak scaling)."""
    return world * 1000.0 / ms_per_step
