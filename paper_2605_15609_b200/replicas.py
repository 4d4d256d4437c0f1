"""Multi-GPU plumbing: independent replicas, one process per GPU.

The PSD step has no exchange between sequences: blocks are independent problems and the LM-head
weights are read-only, so the path shards over GPUs as replicas (each rank holds W and its own
batch of blocks) with no data-path collective.  torch.distributed is used only to line the ranks
up (barrier) and to reduce the timings (max over ranks) and unit counts (sum).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class RankInfo:
    rank: int
    local_rank: int
    world_size: int

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def rank_info_from_env(env=None) -> RankInfo:
    env = os.environ if env is None else env
    return RankInfo(int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", env.get("RANK", "0"))),
                    int(env.get("WORLD_SIZE", "1")))


def init_process_group(info: RankInfo, backend: str | None = None, env=None):
    """Joins the job's process group (no-op for a single process).  NCCL on GPUs, gloo otherwise."""
    if info.world_size <= 1:
        return False
    if dist.is_initialized():
        return True
    env = os.environ if env is None else env
    env.setdefault("MASTER_ADDR", "127.0.0.1")
    env.setdefault("MASTER_PORT", "29500")
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    dist.init_process_group(backend=backend, rank=info.rank, world_size=info.world_size)
    return True


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's own batch of blocks (rank 0 keeps the single-GPU workload)."""
    return base_seed + 1000 * rank


def barrier(info: RankInfo, device=None):
    if info.world_size > 1:
        if device is not None and torch.device(device).type == "cuda":
            dist.barrier(device_ids=[torch.device(device).index])
        else:
            dist.barrier()


def max_over_ranks(value: float, info: RankInfo, device="cpu") -> float:
    if info.world_size <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, info: RankInfo, device="cpu") -> float:
    if info.world_size <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, info: RankInfo, device="cpu"):
    """Whole-job throughput: units of all ranks over the slowest rank's time.  Returns (value, seconds)."""
    secs = max_over_ranks(seconds_this_rank, info, device)
    units = sum_over_ranks(units_this_rank, info, device)
    return units / secs, secs
