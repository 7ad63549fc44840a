"""The step on a tensor-parallel LM head: every rank holds a slice of the vocabulary.

Host plumbing only: how the vocabulary is cut, the two all-gathers, and the order of the three library calls
(`psmc_shard_sweep`, `psmc_shard_locate`, `psmc_shard_finish`).  All arithmetic is in the kernels.

Per step and rank the exchange is 24 bytes per row (a triple of row sums) and then 8 bytes per row (the owner's
token and its logit); the particle state is replicated and stays bit-identical because every rank feeds the same
gathered numbers to the same kernels.
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def vocab_shards(V: int, world: int, align: int = 8) -> List[Tuple[int, int]]:
    """Contiguous (v0, V_local) per rank, tiling [0, V) in rank order.

    Every shard starts on a multiple of `align` columns (8 bf16 or 4 fp32 columns are 16 bytes: the alignment the
    kernels' wide loads and bulk copies need when the whole row is aligned); sizes differ by at most `align`,
    except that the last shard takes the ragged tail.  Every shard gets at least two columns.
    """
    if world < 1 or align < 1 or V < 2 * world:
        raise ValueError("cannot cut %d columns into %d shards" % (V, world))
    units = V // align                      # whole aligned units; the tail (V % align) goes to the last shard
    if units < world:                       # too few aligned units: fall back to unaligned, near-equal shards
        base, extra = divmod(V, world)
        sizes = [base + (1 if r < extra else 0) for r in range(world)]
    else:
        base, extra = divmod(units, world)
        sizes = [(base + (1 if r < extra else 0)) * align for r in range(world)]
        sizes[-1] += V - units * align
    out, v0 = [], 0
    for n in sizes:
        out.append((v0, n))
        v0 += n
    assert v0 == V and all(n >= 2 for _, n in out)
    return out


class Exchange:
    """all_gather(t) -> tensor [world, *t.shape] holding every rank's `t` in rank order."""

    world = 1
    rank = 0

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        return t.unsqueeze(0).clone()


class TorchDistExchange(Exchange):
    """The exchange over a torch.distributed process group (NCCL on GPUs; gloo for host tensors)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist = dist
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self._flat = True

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        out = torch.empty((self.world,) + tuple(t.shape), dtype=t.dtype, device=t.device)
        t = t.contiguous()
        if self._flat:
            try:  # one flat collective straight into `out`
                self._dist.all_gather_into_tensor(out.view(-1), t.view(-1), group=self.group)
                return out
            except (RuntimeError, NotImplementedError):
                self._flat = False  # a backend without it: the list form from now on
        self._dist.all_gather([out[r] for r in range(self.world)], t, group=self.group)
        return out


class VocabShardedStep:
    """One rank's side of the sharded step.

    ps: this rank's `binding.Psmc`, created with the WHOLE vocabulary size and the same parameters and seed on every
    rank.  v0: first column of this rank.  exchange: an `Exchange`.  device: where the exchanged buffers live (the
    current CUDA device unless given).
    """

    def __init__(self, ps, v0: int, exchange: Exchange, device=None):
        self.ps, self.v0, self.ex = ps, int(v0), exchange
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.triples = torch.empty((ps.R, 3), dtype=torch.float64, device=dev)
        self.picks = torch.empty((ps.R, 2), dtype=torch.int32, device=dev)

    def step(self, logits_local: torch.Tensor) -> None:
        """logits_local: CUDA [R, V_local], this rank's columns of the step's logits.

        Kernels and collectives are all issued on torch's current stream, so they are ordered without events.
        """
        ps, ex = self.ps, self.ex
        ps.shard_sweep(logits_local, self.triples)
        all_triples = ex.all_gather(self.triples)
        ps.shard_locate(self.v0, all_triples, ex.rank, self.picks)
        all_picks = ex.all_gather(self.picks)
        ps.shard_finish(all_triples, all_picks)
