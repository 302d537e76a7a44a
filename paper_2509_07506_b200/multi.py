"""Host-side helpers for running on several GPUs, one process per GPU.

All three operations are independent per row (per token), so a batch is sharded by contiguous row
blocks and every rank works on its own block with no collective on the data path.  The only
communication is the timing reduction (max over ranks) that a benchmark or a scheduler needs.
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_rows(total_rows: int, world: int, rank: int) -> Tuple[int, int]:
    """(first_row, row_count) of `rank`'s contiguous block; blocks differ by at most one row,
    cover [0, total_rows) exactly once, and are empty only when there are fewer rows than ranks."""
    if world < 1 or not 0 <= rank < world or total_rows < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(total_rows, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(backend: str, device: torch.device | None = None) -> None:
    """Rendezvous over 127.0.0.1 unless MASTER_ADDR says otherwise."""
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    if backend == "nccl" and device is not None:
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)


def max_over_ranks(values: Sequence[float], device: torch.device | str = "cpu") -> List[float]:
    """Elementwise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_rate(units_per_rank_per_step: float, world: int, steps: int, elapsed_ms: float) -> float:
    """Whole-job rate: units all ranks processed in `steps` steps divided by the (max-over-ranks) time."""
    return world * units_per_rank_per_step * steps / (elapsed_ms * 1e-3)
