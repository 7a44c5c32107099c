"""Host-side bookkeeping for running the path as independent replicas, one per GPU.

The method has no exchange step: every rank runs the whole path on its own copy of
the workload.  The only communication is around the timed region (a barrier before
and after, and the maximum over ranks of the device-side timings), and the job's
throughput is the work of all replicas over the slowest replica's time.
Holds no arithmetic of the method; works with any torch.distributed backend (NCCL
on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class RankInfo:
    rank: int
    local_rank: int
    world: int


def rank_info(env=None) -> RankInfo:
    """Reads the launcher's environment (torch.distributed.run sets these); a plain run is rank 0 of 1."""
    env = os.environ if env is None else env
    return RankInfo(int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0")), int(env.get("WORLD_SIZE", "1")))


def init(info: RankInfo, backend: str, device=None) -> None:
    if info.world <= 1:
        return
    import torch.distributed as dist

    if dist.is_initialized():
        return
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)


def shutdown(info: RankInfo) -> None:
    if info.world <= 1:
        return
    import torch.distributed as dist

    if dist.is_initialized():
        dist.destroy_process_group()


def barrier(info: RankInfo, device=None) -> None:
    """All replicas reach this point; on a GPU also drains the device's queue."""
    if info.world > 1:
        import torch.distributed as dist

        dist.barrier()
    if device is not None and torch.device(device).type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(info: RankInfo, values, device=None):
    """Element-wise maximum over the replicas of a short list of timings."""
    vals = [float(x) for x in values]
    if info.world <= 1:
        return vals
    import torch.distributed as dist

    t = torch.tensor(vals, dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def job_throughput(info: RankInfo, units_per_replica: float, slowest_seconds: float) -> float:
    """Units all replicas processed over the slowest replica's time (weak scaling)."""
    if slowest_seconds <= 0.0:
        raise ValueError("non-positive time")
    return info.world * float(units_per_replica) / float(slowest_seconds)
