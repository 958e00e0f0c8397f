"""Layer-parallel sharding of a quantisation job over ranks.

The method quantises every linear layer on its own (Sec. 3.5: layers are processed
independently), so a multi-GPU job needs no data-path collective: every rank runs the whole
per-layer path on its own layers.  This module holds the host logic of that: which layers a rank
takes, and how per-rank timings combine into a whole-job figure (the slowest rank defines the
step).  It works on any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def layers_for_rank(n_layers: int, rank: int, world: int) -> list[int]:
    """Strong scaling: indices of the layers rank `rank` quantises out of `n_layers` (round-robin,
    so that large and small layers of a decoder stack spread evenly)."""
    if not 0 <= rank < world:
        raise ValueError("rank outside the world")
    return list(range(rank, n_layers, world))


def seed_for_rank(base_seed: int, rank: int) -> int:
    """Weak scaling: every rank draws its own batch of synthetic layers."""
    return base_seed + rank


def max_over_ranks(ms: float, device: torch.device | str = "cpu") -> float:
    """Time of a step of the whole job: the slowest rank's (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(weights_per_rank_step: Sequence[int] | int, rounds: int, ms_step: float, world: int) -> float:
    """Whole-job Gweights/s per k-means round: all ranks' weights x rounds over the step time."""
    total = weights_per_rank_step * world if isinstance(weights_per_rank_step, int) else sum(weights_per_rank_step)
    return total * rounds / (ms_step * 1e-3) / 1e9
