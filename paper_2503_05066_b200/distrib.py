"""Multi-process plumbing for the benchmark: one process per GPU, no collective on the data path.

The layer shards by data-parallel replicas (each rank runs its own batch through its own copy of
the layer), so the only communication is what the measurement needs: a barrier on both sides of
the timed region and a MAX reduction of the per-rank device times.  The same helpers run on the
`gloo` backend for CPU tests.
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Optional

import torch
import torch.distributed as dist


@dataclass
class RankInfo:
    rank: int
    world: int
    local_rank: int


def rank_info_from_env() -> RankInfo:
    return RankInfo(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                    int(os.environ.get("LOCAL_RANK", "0")))


def init(info: RankInfo, backend: str = "nccl", device: Optional[torch.device] = None) -> None:
    if info.world <= 1 or dist.is_initialized():
        return
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = device
    dist.init_process_group(backend, rank=info.rank, world_size=info.world, **kw)


def barrier(info: RankInfo) -> None:
    if info.world > 1:
        dist.barrier()


def max_over_ranks(v: float, info: RankInfo, device: Optional[torch.device] = None) -> float:
    """Every rank gets the largest v."""
    if info.world <= 1:
        return float(v)
    t = torch.tensor([float(v)], dtype=torch.float64, device=device or torch.device("cpu"))
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_seed(base_seed: int, info: RankInfo) -> int:
    """Each replica draws its own batch: distinct, reproducible seeds per rank."""
    return int(base_seed) + info.rank


def job_throughput(units_per_rank: int, ms_per_step_max: float, info: RankInfo) -> float:
    """Whole-job units/s: all ranks' units over the slowest rank's time (weak scaling)."""
    return info.world * units_per_rank / (ms_per_step_max * 1e-3)


def finish(info: RankInfo) -> None:
    if info.world > 1 and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
