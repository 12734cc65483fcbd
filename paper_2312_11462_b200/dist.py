"""Replica aggregation for runs on several GPUs.

The review step of one sequence does not shard without per-layer exchanges, so several GPUs run
independent replicas (one sequence each): no data-path collective.  The only communication is
the max-over-ranks of the measured times, done here with torch.distributed (NCCL on GPUs; the
CPU tests use gloo)."""
from __future__ import annotations

from typing import Optional, Tuple


def aggregate_tokens_per_s(tokens_per_rank: int, device_ms: float, bracket_ms: float, steps: int,
                           dist=None) -> Tuple[float, float, float]:
    """Returns (tokens/s from device time, tokens/s from the bracketed end-to-end time, ms per
    step), each over the whole job: tokens of all ranks divided by the slowest rank's time."""
    world = 1
    if dist is not None:
        import torch
        world = dist.get_world_size()
        dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
        t = torch.tensor([device_ms, bracket_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        device_ms, bracket_ms = float(t[0]), float(t[1])
    total = tokens_per_rank * world
    return total / (device_ms * 1e-3), total / (bracket_ms * 1e-3), bracket_ms / max(steps, 1)


def replica_prompt_seed(base: int, rank: int) -> int:
    """Each replica decodes its own prompt."""
    return base + rank
