"""Host-side plumbing for running the path on several GPUs of one node.

The path shards by independent batches: every rank owns its own sequences and its own copy
of the int4 weights, and no step of the path exchanges data between ranks (weak scaling).
The only cross-rank traffic is the barrier around the timed region and the max-reduction of
the measured time, done with torch.distributed (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass
class RankInfo:
    rank: int
    world: int
    local_rank: int

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def rank_info_from_env() -> RankInfo:
    return RankInfo(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                    int(os.environ.get("LOCAL_RANK", "0")))


def init(info: RankInfo, backend: str | None = None) -> None:
    """Joins the process group (rendezvous via MASTER_ADDR / MASTER_PORT) when world > 1."""
    if info.world <= 1 or dist.is_initialized():
        return
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    dist.init_process_group(backend=backend, rank=info.rank, world_size=info.world)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


def batch_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own batch: same recipe, different seed."""
    return base_seed + 1000 * rank


def barrier(device=None) -> None:
    if dist.is_initialized():
        if device is not None and torch.device(device).type == "cuda":
            dist.barrier(device_ids=[torch.device(device).index or 0])
        else:
            dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's figure (timings are reported as the max over ranks)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> tuple[float, float]:
    """Whole-job throughput: units all ranks processed / slowest rank's time."""
    total_units = sum_over_ranks(units_this_rank, device)
    t = max_over_ranks(seconds_this_rank, device)
    return total_units / t if t > 0 else 0.0, t
