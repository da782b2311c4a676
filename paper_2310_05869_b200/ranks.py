"""One process per GPU: the host-side plumbing of a multi-rank run.

The forward pass shards by (batch, head) segments with no exchange between them, so a run on
N ranks is N independent workloads ("weak" scaling): every rank generates its own segments,
the ranks meet only at a barrier on both sides of the timed region, and the job's time is the
maximum over ranks of the device time.  Nothing here touches the data path; the module works
with any `torch.distributed` backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import dataclasses
import os

from . import workloads as WL


@dataclasses.dataclass(frozen=True)
class RankInfo:
    rank: int
    local_rank: int
    world: int


def rank_env(env=None) -> RankInfo:
    """Rank, local rank and world size as torchrun exports them (a single process otherwise)."""
    env = os.environ if env is None else env
    return RankInfo(int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0")), int(env.get("WORLD_SIZE", "1")))


def init(info: RankInfo, backend: str, device=None):
    """Joins the process group (no-op for a single process).  Rendezvous comes from MASTER_ADDR /
    MASTER_PORT in the environment."""
    if info.world == 1:
        return
    import torch.distributed as dist
    kwargs = {"device_id": device} if (device is not None and backend == "nccl") else {}
    dist.init_process_group(backend, rank=info.rank, world_size=info.world, **kwargs)


def shutdown(info: RankInfo):
    if info.world == 1:
        return
    import torch.distributed as dist
    dist.destroy_process_group()


def rank_workload(w: WL.Workload, rank: int) -> WL.Workload:
    """The workload a rank runs: the same shape, its own input stream (rank 0 keeps the
    single-process workload bit for bit)."""
    return w.scaled(gen_seed=w.gen_seed + 7919 * rank)


def barrier(info: RankInfo):
    if info.world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(info: RankInfo, value: float, device="cpu") -> float:
    """The largest of the ranks' values (every rank receives it)."""
    if info.world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(info: RankInfo, units_per_rank_step: float, steps: int, ms_max: float) -> float:
    """Whole-job units per second: what all ranks processed divided by the slowest rank's time."""
    return units_per_rank_step * steps * info.world / (ms_max * 1e-3)
