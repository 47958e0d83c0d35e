"""Multi-GPU plumbing for the benchmark: one process per GPU, no data-path collective.

The indexer path shards without any exchange (query rows are independent given K, decode
sequences are independent), so ranks run independent problems ("weak" scaling). The only
communication is for measurement: a barrier around the timed region and a MAX-reduce of the
per-rank device time. The same helpers run on CPU with the gloo backend in the tests.
"""
from __future__ import annotations

import os

import torch


def env_rank_world():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT."""
    import torch.distributed as dist
    rank, world, _ = env_rank_world()
    if world > 1 and not dist.is_initialized():
        kwargs = {}
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend, rank=rank, world_size=world, **kwargs)
    return rank, world


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    """The slowest rank's time: what a whole-job throughput must be divided by."""
    if world == 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the independent problem a rank works on."""
    return base_seed + 1000 * rank


def whole_job_rate(units_per_rank: float, steps: int, slowest_ms: float, world: int) -> float:
    """Units processed by all ranks per second."""
    return world * units_per_rank * steps / (slowest_ms * 1e-3)


def shutdown(world: int):
    if world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
