"""Multi-GPU plumbing of the benchmark: one process per GPU, independent sequences per rank.

The ATP path shards across sequences (every sequence has its own basis and attention), so the data
path needs no collective. torch.distributed is used for two things only: a barrier around the timed
region and the maximum of the per-rank device times. The same code runs on the gloo backend on CPU,
which is how it is tested without GPUs.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    """(world_size, rank, local_rank) from the launcher's environment (1, 0, 0 when run directly)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> Tuple[int, int]:
    """Join the process group named by the environment; returns (world_size, rank)."""
    world, rank, _ = env_ranks()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return world, rank


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own sequences: weak scaling over independent problems."""
    return base_seed + 17 * rank


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's time: the job's time."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, steps: int, ms_max: float, world: int) -> float:
    """Whole-job throughput: tokens of all ranks over the slowest rank's time."""
    return world * tokens_per_rank * steps / (ms_max / 1e3)


def finish():
    if dist.is_initialized():
        dist.destroy_process_group()
