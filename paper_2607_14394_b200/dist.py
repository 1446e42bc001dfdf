"""Host-side plumbing for running the layer on several GPUs of one node.

The spectral layer partitions over independent samples: each rank owns its own
slice of the global batch and runs the whole path on it with no data-path
collective (weak scaling).  Only the timing is reduced (max over ranks).
"""
from __future__ import annotations

import os
from typing import Sequence


def env_world():
    """(world_size, rank, local_rank) from the torchrun environment (defaults: single process)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(backend: str, device=None):
    """Joins the default process group when WORLD_SIZE > 1; rendezvous on 127.0.0.1 unless told otherwise."""
    import torch.distributed as dist
    world, _, _ = env_world()
    if world <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    if backend == "nccl" and device is not None:
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)
    return True


def batch_shard(global_batch: int, world: int, rank: int):
    """Contiguous [start, stop) of the samples rank `rank` owns; sizes differ by at most one."""
    if not (0 <= rank < world) or global_batch < 0:
        raise ValueError("bad rank/world/batch")
    base, extra = divmod(global_batch, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def rank_seed(seed: int, rank: int) -> int:
    """Distinct, reproducible input seed per rank."""
    return int(seed) * 1009 + int(rank)


def max_over_ranks(values: Sequence[float], device="cpu"):
    """Element-wise max over all ranks of a short list of floats (timings)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def sum_over_ranks(value: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t[0])


def whole_job_throughput(points_per_rank_step: Sequence[float] | float, ms_per_step_max: float, world: int) -> float:
    """Whole-job grid points per second: every rank's points over the slowest rank's step time."""
    total = float(points_per_rank_step) * world if not isinstance(points_per_rank_step, (list, tuple)) \
        else float(sum(points_per_rank_step))
    return total / (ms_per_step_max * 1e-3)
