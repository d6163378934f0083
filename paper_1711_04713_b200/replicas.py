"""Host-side helpers for data-parallel replicas (one process per GPU, batch sharded, weights
replicated).  The forward path itself needs no exchange; only calibration does: every replica must
fix the same decimal point per layer, so the per-layer range (one int64) is max-reduced, and the
sparsity / saturation counters (three uint64) are sum-reduced for reporting.  Works on any
torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own images: distinct, reproducible streams."""
    return int(base_seed) + int(rank)


def agree_on_range(max_abs_acc: int, device="cpu", group=None) -> int:
    """Largest per-layer range over all replicas (max-reduce of one int64)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return int(max_abs_acc)
    t = torch.tensor([int(max_abs_acc)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return int(t[0])


def sum_counters(zeros: int, sat_pos: int, sat_neg: int, device="cpu", group=None) -> tuple[int, int, int]:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return int(zeros), int(sat_pos), int(sat_neg)
    t = torch.tensor([int(zeros), int(sat_pos), int(sat_neg)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return int(t[0]), int(t[1]), int(t[2])


def largest_float(value: float, device="cpu", group=None) -> float:
    """Largest value over all replicas (the input's max |x| during calibration)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float32, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t[0])


def sum_histogram(hist, device="cpu", group=None) -> list[int]:
    """Bin-wise sum of a bit-occupancy histogram over all replicas (thresholded allocation)."""
    hist = [int(v) for v in hist]
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return hist
    t = torch.tensor(hist, dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return [int(v) for v in t.tolist()]


def slowest_rank_ms(elapsed_ms: float, device="cpu", group=None) -> float:
    """A multi-GPU step takes as long as its slowest replica."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(elapsed_ms)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t[0])


def whole_job_rate(units_per_rank: int, world_size: int, ms_per_step: float) -> float:
    """Units (images) per second over all replicas."""
    return world_size * units_per_rank / (ms_per_step / 1e3)
