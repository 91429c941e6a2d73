"""Process-group plumbing for running the step on N GPUs (one process per GPU).

Replicas: the gradient step has no exchange between GPUs when each GPU emulates its own K
workers, so N GPUs run N replicas and the only collectives are the barrier and the
max-over-ranks of the timings. Parameter shards of ONE problem (ShardedDmx) have one exchange
step: the sum of the shards' raw fp64 sums (`allreduce_sum`).
"""
from __future__ import annotations

import os

_world = 1
_group = False      # a process group exists: the collectives run (always so when the world has more than one rank)


def init(world: int, backend: str = "nccl", group_of_one: bool = False) -> None:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT.
    A world of one needs no group and every collective below is then the identity; with
    `group_of_one` a one-rank group is created all the same and the collectives run through the
    backend (how the nccl branches are exercised where only one GPU is available)."""
    global _world, _group
    _world = int(world)
    _group = _world > 1 or group_of_one
    if not _group:
        return
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=int(os.environ.get("RANK", "0")), world_size=_world)


def _host_staged():
    """gloo moves host memory: device tensors go through a host copy (tests on CPU or with
    several processes on one GPU); nccl takes device tensors as they are."""
    import torch.distributed as dist
    return dist.get_backend() != "nccl"


def barrier() -> None:
    if _group:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float) -> float:
    """Max of a per-rank scalar (timings are reported as the slowest rank's)."""
    if not _group:
        return float(x)
    import torch
    import torch.distributed as dist
    dev = "cpu" if _host_staged() else "cuda"
    t = torch.tensor([float(x)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def allreduce_sum(t):
    """Entry-wise sum over the ranks of a tensor (the shards' partial sums), in place; the
    tensor lives where the backend wants it (device memory for nccl, host memory for gloo)."""
    if _group:
        import torch.distributed as dist
        if _host_staged() and t.is_cuda:
            h = t.cpu()
            dist.all_reduce(h, op=dist.ReduceOp.SUM)
            t.copy_(h)
        else:
            dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def shard_ranges(P: int, world: int):
    """[(lo, hi)] of the `world` parameter shards (the library's own split)."""
    from . import binding as B
    out = []
    for r in range(world):
        rc, lo, hi = B.dmx_shard_range(P, world, r)
        if rc != B.OK:
            raise B.DmxError(rc, "dmx_shard_range")
        out.append((lo, hi))
    return out


def exchange_gradient_ranges(local_grad, ranges, rank: int):
    """Worker k is rank k and holds its own gradient (P elements). Returns a (world, stride)
    tensor whose row k holds worker k's values of THIS rank's parameter range [lo, hi) in its
    first hi - lo entries (stride = that length rounded up to 8 elements, so that every row
    starts on a 16-byte boundary). Every worker's values are needed, not their sum: the
    per-worker norms and the spread across workers are computed from them. One all-to-all
    (nccl); gloo, which has none, gathers the whole gradients and slices (tests only)."""
    import torch
    import torch.distributed as dist
    world = len(ranges)
    lo, hi = ranges[rank]
    n = hi - lo
    stride = (n + 7) // 8 * 8
    out = torch.zeros((world, max(stride, 8)), dtype=local_grad.dtype, device=local_grad.device)
    if not _group:
        out[0, :n] = local_grad[lo:hi]
        return out
    if not _host_staged():
        send = [local_grad[a:b] for a, b in ranges]
        recv = [out[k, :n] for k in range(world)]
        dist.all_to_all(recv, send)
    else:
        mine = local_grad.contiguous().cpu()
        full = [torch.empty_like(mine) for _ in range(world)]
        dist.all_gather(full, mine)
        for k in range(world):
            out[k, :n] = full[k][lo:hi].to(out.device)
    return out


def gather_batch_sizes(b_local: int):
    """Every worker's batch size, in rank order (host ints)."""
    if not _group:
        return [int(b_local)]
    import torch
    import torch.distributed as dist
    dev = "cpu" if _host_staged() else "cuda"
    mine = torch.tensor([int(b_local)], dtype=torch.int64, device=dev)
    every = [torch.zeros_like(mine) for _ in range(_world)]
    dist.all_gather(every, mine)
    return [int(t.item()) for t in every]


def allgather_ranges(shard, ranges, out_full):
    """Rebuild a whole-length vector (the updated parameters) from the ranks' shards: out_full[lo_r:hi_r] =
    rank r's shard. Shards differ in length, so instead of one all-gather of padded copies every rank's
    shard is broadcast straight into its place in `out_full` (one broadcast per non-empty shard, all in
    flight together): each byte crosses the link once and nothing is staged on the device."""
    import torch
    import torch.distributed as dist
    if not _group:
        out_full[ranges[0][0]:ranges[0][1]] = shard[:ranges[0][1] - ranges[0][0]]
        return out_full
    me = dist.get_rank()
    staged = _host_staged() and out_full.is_cuda
    dst = torch.empty(out_full.numel(), dtype=out_full.dtype, device="cpu") if staged else out_full
    a, b = ranges[me]
    dst[a:b] = shard[:b - a].to(dst.device)
    works = [dist.broadcast(dst[lo:hi], src=r, async_op=True) for r, (lo, hi) in enumerate(ranges) if hi > lo]
    for w in works:
        w.wait()
    if staged:
        out_full.copy_(dst)
    return out_full


def worker_per_gpu_step(sh, rank, ranges, local_grad, b_local, params_shard, momentum_shard, prev_shard, lr, beta,
                        params_full=None):
    """One step with worker k on GPU k (K = world size) and the model state sharded by parameter
    range: gather the batch sizes, exchange gradient ranges, run the fused pass on this rank's
    shard (ShardedDmx `sh`, created with nshards = world, shard = rank), add the partial sums over
    the ranks, derive the state vector (identical on every rank), and optionally rebuild the full
    parameter vector. Returns the state vector."""
    b = gather_batch_sizes(b_local)
    rows = exchange_gradient_ranges(local_grad, ranges, rank)
    part = sh.step_partial([rows[k] for k in range(len(ranges))], b, params_shard, momentum_shard, lr, beta, prev_shard,
                           local=True)
    allreduce_sum(part)
    state = sh.finalize(b, part)
    if params_full is not None:
        allgather_ranges(params_shard, ranges, params_full)
    return state


def job_throughput(units_per_rank: float, local_ms: float) -> float:
    """Whole-job units per second of N replicas: N * units / slowest rank's time."""
    return _world * units_per_rank / (max_over_ranks(local_ms) * 1e-3)


def finish() -> None:
    global _world, _group
    if _group:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.barrier()
            dist.destroy_process_group()
    _world = 1
    _group = False
