"""Rank plumbing for running independent replicas of the hot path, one process per GPU.

The path shards by sequence with no exchange step (compression is independent per prompt and
KV head, decode attention per sequence), so N GPUs simply hold N disjoint sets of sequences.
The only cross-rank operations are the ones a benchmark needs: a barrier around the timed
region and the maximum of the per-rank times.  Nothing here touches the data path.
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Optional

import torch
import torch.distributed as dist


@dataclass
class ReplicaGroup:
    rank: int
    world: int
    local_rank: int
    backend: Optional[str]

    @property
    def is_root(self) -> bool:
        return self.rank == 0

    def seed_for(self, base_seed: int, stride: int = 1000) -> int:
        """Distinct, reproducible input seed per replica."""
        return int(base_seed) + stride * self.rank

    def barrier(self) -> None:
        if self.world > 1:
            dist.barrier()

    def max_over_ranks(self, value: float, device="cpu") -> float:
        """Largest value over all replicas (the time of the slowest rank)."""
        if self.world == 1:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, value: float, device="cpu") -> float:
        """Total over all replicas (units of work processed by the whole job)."""
        if self.world == 1:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def aggregate_throughput(self, units_this_rank: float, elapsed_ms_this_rank: float, device="cpu"):
        """Whole-job throughput: all units processed divided by the slowest rank's time.
        Returns (units per second, max elapsed ms)."""
        ms = self.max_over_ranks(elapsed_ms_this_rank, device)
        units = self.sum_over_ranks(units_this_rank, device)
        return units / (ms * 1e-3), ms

    def close(self) -> None:
        if self.world > 1 and dist.is_initialized():
            dist.destroy_process_group()


def init_from_env(backend: Optional[str] = None, device=None) -> ReplicaGroup:
    """Reads RANK / WORLD_SIZE / LOCAL_RANK / MASTER_* as set by torchrun; with one process no
    process group is created.  backend: "nccl" on GPUs, "gloo" for CPU-only runs."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        be = backend or ("nccl" if torch.cuda.is_available() else "gloo")
        kw = {}
        if be == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(be, rank=rank, world_size=world, **kw)
        backend = be
    return ReplicaGroup(rank, world, local, backend if world > 1 else None)
