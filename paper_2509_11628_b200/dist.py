"""Process-group plumbing for running one independent cache per GPU.

The path shards by sample batch with no exchange step: every rank owns its own batch of samples
and its own cache, so the only collectives are the barrier around the timed region and the
max-over-ranks of the measured time. Works with ``nccl`` (GPU) and ``gloo`` (CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import List, Sequence

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


def init(backend: str) -> RankInfo:
    """Join the process group described by the torchrun environment (no-op for one process)."""
    info = rank_info_from_env()
    if info.world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=info.rank, world_size=info.world)
    return info


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The slowest rank's time: what a multi-GPU number must be quoted on."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def combine_verify_sums(sums: torch.Tensor, linf: bool = False) -> torch.Tensor:
    """Token-sharded verification: combine every rank's per-sample running values ([B, 4] float64, as
    speca_verify_partial writes them) in place -- a sum, or a maximum for the l-infinity metric. This
    is the path's only exchange step in that layout: 32 bytes per sample per speculative step. A NaN
    in any shard must survive the maximum, so NaNs are counted separately and put back."""
    if not dist.is_initialized():
        return sums
    if linf:
        nan = torch.isnan(sums).to(sums.dtype)
        clean = torch.nan_to_num(sums, nan=0.0)
        dist.all_reduce(clean, op=dist.ReduceOp.MAX)
        dist.all_reduce(nan, op=dist.ReduceOp.MAX)
        sums.copy_(torch.where(nan > 0, torch.full_like(clean, float("nan")), clean))
    else:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM)
    return sums


def shard_tokens(n_tokens: int, world: int, rank: int):
    """(first token, count) of this rank's contiguous token range; sizes differ by at most one."""
    base, extra = divmod(n_tokens, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def shard_samples(n_samples: int, world: int, rank: int) -> List[int]:
    """Contiguous, balanced split of global sample indices over ranks (sizes differ by at most 1)."""
    base, extra = divmod(n_samples, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def gather_decisions(local_accept: Sequence[int], device: str = "cpu") -> List[List[int]]:
    """Every rank's per-sample accept flags, for a scheduler that wants the global picture. The data
    path itself never needs this: a sample's decision depends on that sample alone."""
    if not dist.is_initialized():
        return [list(local_accept)]
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, list(local_accept))
    return out
