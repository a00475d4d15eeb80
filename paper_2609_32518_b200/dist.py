"""Multi-process plumbing for one-process-per-GPU runs.

The chunk-attention path has no exchange step: streams (and heads) are independent, so
N GPUs run N independent shards and nothing crosses NVLink on the data path.  What is
shared is bookkeeping only: a barrier around the timed region, the max of a time over
the ranks and the split of streams or heads over ranks.  NCCL on GPUs, gloo on CPU (tests)."""

from __future__ import annotations

import os


def env_ranks():
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None, device=None) -> tuple:
    """Join the process group when WORLD_SIZE > 1.  Returns (rank, local_rank, world)."""
    import torch.distributed as dist
    rank, local_rank, world = env_ranks()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kwargs = {}
        if backend is None:
            backend = "nccl" if device is not None and getattr(device, "type", "") == "cuda" else "gloo"
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend, rank=rank, world_size=world, **kwargs)
    return rank, local_rank, world


def finalize():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def barrier(device=None):
    """Process barrier; with a CUDA device also drains that device on both sides."""
    import torch
    import torch.distributed as dist
    if device is not None and getattr(device, "type", "") == "cuda":
        torch.cuda.synchronize(device)
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
    if device is not None and getattr(device, "type", "") == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a host float over all ranks (the job's time is its slowest rank's)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64,
                     device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_streams(n_streams: int, rank: int, world: int) -> range:
    """Contiguous, balanced split of independent streams over ranks (no stream is split)."""
    lo = n_streams * rank // world
    hi = n_streams * (rank + 1) // world
    return range(lo, hi)


def shard_heads(n_heads: int, rank: int, world: int) -> range:
    """Contiguous, balanced split of the attention heads over ranks.  Heads never interact, so a
    rank that owns heads [lo, hi) keeps the cache slices [B, C, T, hi - lo, 128] of those heads,
    appends and attends them alone, and its output is the [.., lo:hi, :] slice of the whole
    output: no exchange inside the path (12 heads -> 2, 3, 4 or 6 GPUs; 40 heads -> 8 x 5)."""
    lo = n_heads * rank // world
    hi = n_heads * (rank + 1) // world
    return range(lo, hi)
