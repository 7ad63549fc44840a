"""Running the path on several GPUs: independent replicas, one process per GPU.

Prompts (groups) never exchange anything in Algorithm 1, so the path shards by prompt with no
data-path collective: every rank owns its own prompts, its own caches and its own random stream.
The only communication is bookkeeping around a measurement: a barrier, the slowest rank's device
time and the total number of particle-tokens.  These helpers hold that host logic so that it can be
exercised on CPU (`gloo`) as well as on GPUs (`nccl`).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class RankPlan:
    rank: int
    world: int
    local_rank: int
    seed: int          # seed of this rank's prompts: ranks draw different prompts and uniforms
    group_offset: int  # index of this rank's first prompt in the whole job's numbering


def rank_plan(groups_per_rank: int, base_seed: int = 1, env=None) -> RankPlan:
    """Who am I and which prompts are mine.  Weak scaling: every rank carries `groups_per_rank` prompts."""
    env = os.environ if env is None else env
    world = int(env.get("WORLD_SIZE", "1"))
    rank = int(env.get("RANK", "0"))
    local = int(env.get("LOCAL_RANK", "0"))
    if not (0 <= rank < world):
        raise ValueError("RANK %d outside WORLD_SIZE %d" % (rank, world))
    return RankPlan(rank, world, local, base_seed + rank, rank * groups_per_rank)


def shard_groups(n_groups: int, world: int, rank: int):
    """Strong-scaling split of a fixed set of prompts: contiguous, sizes differing by at most one."""
    if world < 1 or not (0 <= rank < world) or n_groups < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_groups, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def _reduce(x: float, op, device) -> float:
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float, device="cpu") -> float:
    import torch.distributed as dist
    return _reduce(x, dist.ReduceOp.MAX, device)


def sum_over_ranks(x: float, device="cpu") -> float:
    import torch.distributed as dist
    return _reduce(x, dist.ReduceOp.SUM, device)


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def job_throughput(units_local: float, ms_local: float, device="cpu"):
    """Whole-job rate: units processed by all ranks / the slowest rank's device time.  Returns (rate per second,
    ms of the slowest rank, total units)."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_local, device)
    return units / (ms * 1e-3), ms, units
