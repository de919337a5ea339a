"""Replica bookkeeping for multi-GPU runs.

The compression path has no exchange step (every cache, layer and KV head is an
independent problem), so N GPUs run N independent replicas: one process per
GPU, no data-path collective.  The only communication is the benchmark's own
bookkeeping: a barrier around the timed region, the maximum of the per-rank
device times and the sum of the per-rank work.  Works unchanged with one
process and no process group.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as td


def init(backend: str) -> None:
    if td.is_available() and not td.is_initialized() and int(os.environ.get("WORLD_SIZE", "1")) > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        td.init_process_group(backend=backend)


def _active() -> bool:
    return td.is_available() and td.is_initialized() and td.get_world_size() > 1


def _device() -> torch.device:
    return torch.device("cuda", torch.cuda.current_device()) if td.get_backend() == "nccl" else torch.device("cpu")


def world_size() -> int:
    return td.get_world_size() if _active() else 1


def barrier() -> None:
    if _active():
        td.barrier()


def max_over_ranks(x: float) -> float:
    if not _active():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    td.all_reduce(t, op=td.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float) -> float:
    if not _active():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    td.all_reduce(t, op=td.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units: float, elapsed_ms: float) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return sum_over_ranks(units) / (max_over_ranks(elapsed_ms) * 1e-3)


def finish() -> None:
    if td.is_available() and td.is_initialized():
        td.destroy_process_group()
