"""Process-group plumbing for running the step on N GPUs (one process per GPU).

Replicas: the gradient step has no exchange between GPUs when each GPU emulates its own K
workers, so N GPUs run N replicas and the only collectives are the barrier and the
max-over-ranks of the timings. Parameter shards of ONE problem (ShardedDmx) have one exchange
step: the sum of the shards' raw fp64 sums (`allreduce_sum`).
"""
from __future__ import annotations

import os

_world = 1


def init(world: int, backend: str = "nccl") -> None:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT."""
    global _world
    _world = int(world)
    if _world <= 1:
        return
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=int(os.environ["RANK"]), world_size=_world)


def barrier() -> None:
    if _world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float) -> float:
    """Max of a per-rank scalar (timings are reported as the slowest rank's)."""
    if _world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(x)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def allreduce_sum(t):
    """Entry-wise sum over the ranks of a tensor (the shards' partial sums), in place; the
    tensor lives where the backend wants it (device memory for nccl, host memory for gloo)."""
    if _world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def job_throughput(units_per_rank: float, local_ms: float) -> float:
    """Whole-job units per second of N replicas: N * units / slowest rank's time."""
    return _world * units_per_rank / (max_over_ranks(local_ms) * 1e-3)


def finish() -> None:
    global _world
    if _world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.barrier()
            dist.destroy_process_group()
    _world = 1
