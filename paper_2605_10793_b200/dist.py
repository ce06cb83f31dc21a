"""Process-group plumbing for multi-GPU runs (one process per GPU, launched by torchrun).

By default N > 1 means N independent replicas (one context = one GPU, no data-path collective): the only
communication is the barrier around a timed region and a max-reduction of the measured time; independent problems
(the per-head variant) are split over the ranks without any exchange.  `TokenSharded` is the one place with a
data-path collective: one rotation calibrated on token shards, its statistics summed over the ranks before the
update.  Works with NCCL (GPU) and gloo (CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass
class Group:
    rank: int
    local_rank: int
    world: int
    active: bool       # a process group was initialised

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def init(backend: str | None = None) -> Group:
    """Read RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* from the environment; single process if absent."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world <= 1:
        return Group(0, local, 1, False)
    import torch
    import torch.distributed as dist
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if backend == "nccl":
        torch.cuda.set_device(local)
        dist.init_process_group(backend, rank=rank, world_size=world, device_id=torch.device("cuda", local))
    else:
        dist.init_process_group(backend, rank=rank, world_size=world)
    return Group(rank, local, world, True)


def barrier(g: Group) -> None:
    if g.active:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(g: Group, value: float) -> float:
    """The slowest rank's value (timings are reported as the max over ranks)."""
    if not g.active:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(g: Group, value: float) -> float:
    if not g.active:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_problems(n_problems: int, g: Group) -> range:
    """Contiguous block of independent problems owned by this rank (batched / per-head variant)."""
    per = (n_problems + g.world - 1) // g.world
    lo = min(n_problems, g.rank * per)
    return range(lo, min(n_problems, lo + per))


def finish(g: Group) -> None:
    if g.active:
        import torch.distributed as dist
        dist.destroy_process_group()


class TokenSharded:
    """One rotation calibrated on token shards: every rank holds the same R and streams its own rows through its own
    context; at update time the statistics of the Procrustes problem -- the cross-covariance M (d x d) and the
    objective sums J, N, all plain sums over tokens (Sections 3.3-3.4) -- are summed over the ranks with one
    all-reduce each, after which every rank runs the same update on the same M and ends with the same R.

    `ctx` is a single-problem calibration context (step / get_M / set_M / get_objective / update / get_R, as
    binding.Context); with NCCL the all-reduce runs on the context's device tensors.  The sum enters the context
    through conqur_get_M / conqur_set_M, i.e. two extra d x d copies per update.
    The exchange logic is covered by a two-rank gloo test with a CPU stand-in for the context.
    """

    def __init__(self, ctx, g: Group):
        self.ctx, self.g = ctx, g

    def step(self, x_local):
        self.ctx.step(x_local)

    def reduce_statistics(self):
        """All-reduce (sum) M, J, N over the ranks; returns the global (J, N)."""
        j, n = self.ctx.get_objective()
        if not self.g.active:
            return j, n
        import torch
        import torch.distributed as dist
        m = self.ctx.get_M()
        jn = torch.tensor([float(j), float(n)], dtype=torch.float64, device=m.device)
        dist.all_reduce(m, op=dist.ReduceOp.SUM)
        dist.all_reduce(jn, op=dist.ReduceOp.SUM)
        j_tot, n_tot = float(jn[0].item()), int(round(float(jn[1].item())))
        self.ctx.set_M(m, [j_tot], [n_tot])
        return j_tot, n_tot

    def update(self):
        jn = self.reduce_statistics()
        self.ctx.update()
        return jn
