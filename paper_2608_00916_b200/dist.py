"""Multi-GPU plumbing for the benchmark: one process per GPU, data parallel over tokens.

The layer shards over tokens with the experts replicated (expert-parallel degree 1), so the data path needs
no collective; torch.distributed only provides the barrier around the timed region and the max-over-ranks
reduction of its duration.  Works with the gloo backend on CPU (tests) and nccl on GPUs."""
from __future__ import annotations

import os

_state = {"world": 1, "rank": 0, "backend": None}


def init(world: int, rank: int, backend: str = "nccl") -> None:
    _state.update(world=world, rank=rank, backend=backend)
    if world <= 1:
        return
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)


def shard_seed(seed: int, rank: int) -> int:
    """Seed of the token batch drawn by `rank`; rank 0 keeps the workload's own seed."""
    return seed + 7919 * rank


def tokens_per_rank(total_tokens: int, world: int, rank: int) -> int:
    """Strong-scaling split of a fixed batch (not used by the weak-scaling benchmark): balanced, remainder to the
    lowest ranks."""
    base, rem = divmod(total_tokens, world)
    return base + (1 if rank < rem else 0)


def barrier() -> None:
    if _state["world"] > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float) -> float:
    if _state["world"] <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if _state["backend"] == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if _state["world"] <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if _state["backend"] == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(tokens_this_rank: int, ms_this_rank: float) -> float:
    """Whole-job tokens/s: tokens of all ranks over the slowest rank's time."""
    total = sum_over_ranks(tokens_this_rank)
    ms = max_over_ranks(ms_this_rank)
    return total / (ms / 1e3)


def finish() -> None:
    if _state["world"] > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
