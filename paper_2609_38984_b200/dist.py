"""Multi-GPU plumbing: the path shards by sample (independent action chunks), one process per GPU, with no
data-path collective.  Only timing and result reporting cross ranks (a MAX and a SUM all-reduce)."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist

from . import workloads as W


def env_rank() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_rank()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def rank_workload(wl: W.Workload, rank: int, world: int) -> W.Workload:
    """Weak scaling: every rank processes its own batch of `wl.batch` samples, drawn from a rank-specific seed so
    that no two ranks see the same action chunk."""
    if world <= 1:
        return wl
    return wl.with_(seed=wl.seed + 1000 * rank, name=f"{wl.name}@rank{rank}")


def sample_range(n_samples: int, rank: int, world: int) -> range:
    """Strong-scaling split of a fixed set of samples: contiguous, sizes differing by at most one."""
    base, extra = divmod(n_samples, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def barrier(device=None) -> None:
    if dist.is_initialized():
        if device is not None and device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def max_over_ranks(value: float, device=None) -> float:
    if not dist.is_initialized():
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    if not dist.is_initialized():
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def finalize() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
