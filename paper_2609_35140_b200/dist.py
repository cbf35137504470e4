"""Multi-process plumbing for the benchmark: one process per GPU, replicas only.

Attention rows are independent per (sequence, KV head) and log-prob rows per token, so N
GPUs run N independent replicas of the workload with no data-path collective (weak
scaling).  torch.distributed is used only for the barrier around the timed region and for
the max-over-ranks reduction of the measured times.
"""
from __future__ import annotations

import os
from typing import Dict, List

import torch
import torch.distributed as dist


def env_world() -> (int, int, int):
    """(rank, local_rank, world_size) from the torchrun environment (1 process: 0, 0, 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> (int, int, int):
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values: Dict[str, float], device="cpu") -> Dict[str, float]:
    """Element-wise maximum of a dict of floats over all ranks (identity for one process)."""
    if not (dist.is_available() and dist.is_initialized()):
        return dict(values)
    keys = sorted(values)
    t = torch.tensor([values[k] for k in keys], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return {k: float(x) for k, x in zip(keys, t.tolist())}


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def replica_seed_offset(rank: int) -> int:
    """Every replica draws its own tensors (same shapes and length mix, different values)."""
    return 1000003 * rank


def shard_sequences(n_sequences: int, rank: int, world: int) -> List[int]:
    """Contiguous, balanced split of whole sequences across ranks (for callers that want to
    split one batch instead of replicating it; sequences never straddle ranks, so no
    exchange step is needed)."""
    base, extra = divmod(n_sequences, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def finalize() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
