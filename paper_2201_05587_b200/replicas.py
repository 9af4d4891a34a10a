"""Multi-GPU plumbing.  The hot path does not shard: the evaluator's timings are only comparable on one GPU and a
batch-1 model has nothing to split, so N GPUs run N independent replicas.  The only cross-rank traffic is the
barrier around the timed region and two scalar reductions (max of the elapsed time, sum of the work done)."""
from __future__ import annotations

import os


def env_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str):
    """Join the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT; no-op for one process."""
    import torch.distributed as dist
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def _reduce(value: float, op_name: str, device) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, "MAX", device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, "SUM", device)


def aggregate(units_local: float, seconds_local: float, device="cpu"):
    """Whole-job throughput of independent replicas: all units done, divided by the slowest rank's time."""
    total = sum_over_ranks(units_local, device)
    slowest = max_over_ranks(seconds_local, device)
    return total / slowest, slowest


def finalize():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
