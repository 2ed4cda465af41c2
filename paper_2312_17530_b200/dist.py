"""Multi-process plumbing of the benchmark: one process per GPU, no data-path collective.

Every data-parallel rank compresses its own workers' gradients (the path shards by worker),
so ranks only meet at a barrier before/after the timed region and in a MAX reduction of the
elapsed time.  Works with the "nccl" backend on GPUs and with "gloo" on CPU (tests).
"""
from __future__ import annotations

import os
from typing import List, Tuple


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    import torch.distributed as dist

    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def _device_for_backend():
    import torch
    import torch.distributed as dist

    return torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")


def barrier() -> None:
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float) -> float:
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device_for_backend())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float) -> float:
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device_for_backend())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def worker_ids(rank: int, workers_per_rank: int) -> List[int]:
    """Global ids of the simulated workers a rank owns (contiguous blocks, weak scaling)."""
    return list(range(rank * workers_per_rank, (rank + 1) * workers_per_rank))


def aggregate_throughput(units_this_rank: float, elapsed_s_this_rank: float) -> Tuple[float, float]:
    """(whole-job units per second, max elapsed seconds): all ranks' units over the slowest
    rank's time."""
    t = max_over_ranks(elapsed_s_this_rank)
    u = sum_over_ranks(units_this_rank)
    return u / t, t


def finalize() -> None:
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
