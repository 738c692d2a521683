"""Host-side plumbing for running independent replicas of the step, one process per GPU.

The per-sample-weight step does not shard in this library: each rank owns a whole
problem (its own seeded batch and parameter vector) and there is no data-path
collective.  With a shared meta learner (Sec. 4.1) the ranks' dim(lambda)-sized
meta gradients are combined by one all-reduce per meta step (Sec. 3.3, Fig. 2):
all_reduce_sum / all_reduce_mean below.  What the ranks otherwise share is only measurement: a barrier on both sides
of a timed region, the maximum of a duration over ranks, and the aggregate
throughput (units processed by all ranks divided by that maximum).  The same
code runs over NCCL on GPUs and over gloo on CPU (which is how it is tested).
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Optional


@dataclass
class Replicas:
    rank: int
    world: int
    local_rank: int
    backend: Optional[str]  # None when world == 1

    @property
    def seed(self) -> int:
        """Workload seed of this rank: every replica draws an independent problem."""
        return self.rank

    def barrier(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max_over_ranks(self, x: float, device: str = "cpu") -> float:
        if self.world == 1:
            return float(x)
        import torch
        import torch.distributed as dist
        t = torch.tensor([float(x)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def all_reduce_sum(self, t):
        """In-place sum of a tensor over ranks: the one gradient synchronisation of the data-parallel step
        (Sec. 3.3).  With a shared meta learner every rank computes the central difference of Eq. 5 on its own
        rows of the base batch with the whole batch's size as the normaliser (the B_norm argument of
        sama_fd_metagrad_reweight), and this sum of the ranks' dim(lambda)-sized vectors is the batch's meta gradient."""
        if self.world > 1:
            import torch.distributed as dist
            dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t

    def all_reduce_mean(self, t):
        """In-place mean over ranks: for ranks that each ran the whole step on their own batch (and their own direct
        gradient), the way the paper's data-parallel runs average per-replica meta gradients."""
        self.all_reduce_sum(t)
        if self.world > 1:
            t /= self.world
        return t

    def shard_range(self, n: int, align: int = 4):
        """This rank's contiguous share [lo, hi) of a flat vector of n elements, boundaries at multiples of
        ``align`` (16-byte groups for fp32), the remainder going to the last rank.  For running adaptation and
        perturbation on a sharded parameter vector: every rank calls sama_adapt on its share, the ranks'
        sums of squares are added with all_reduce_sum (one double: the norm of Sec. 3.2 is global), and
        sama_perturb takes that sum as its p_sumsq argument."""
        per = (n // self.world) // align * align
        lo = self.rank * per
        hi = n if self.rank == self.world - 1 else lo + per
        return lo, hi

    def aggregate_rate(self, units_per_rank: float, seconds_this_rank: float, device: str = "cpu") -> float:
        """Whole-job throughput: all ranks' units over the slowest rank's time."""
        return self.world * units_per_rank / self.max_over_ranks(seconds_this_rank, device)

    def close(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


def init(backend: str = "nccl", device: Optional[str] = None) -> Replicas:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* from the environment and joins the group."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return Replicas(rank, world, local, None)
    import torch
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = torch.device(device)
    dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return Replicas(rank, world, local, backend)
