"""Multi-process plumbing for runs with one process per GPU.

The sign+vote path has no exchange step when all R buffers of a chunk sit on one
GPU, so N GPUs scan N independent replica sets (weak scaling).  The only
cross-rank work is a barrier around the timed region and the max-over-ranks of
the device time; both go through ``torch.distributed`` (NCCL on GPUs, gloo on
CPU in the tests)."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def rank_info() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> None:
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29513")
    if backend == "nccl":
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def reduce_device() -> str:
    """Where the tensors of the small cross-rank reductions live: the GPU under NCCL."""
    if dist.is_available() and dist.is_initialized() and dist.get_backend() == "nccl":
        return "cuda"
    return "cpu"


def max_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank scans its own replica set."""
    return base_seed + 4096 * rank


def aggregate_gbs(bytes_per_rank: int, world: int, steps: int, ms_max: float) -> float:
    """Whole-job GB/s: the bytes all ranks scanned over the slowest rank's time."""
    return world * bytes_per_rank * steps / (ms_max * 1e-3) / 1e9
