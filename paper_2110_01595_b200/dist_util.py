"""Process-group plumbing for multi-GPU benchmark runs (one process per GPU, no data-path collective).

The path shards as independent problems, so the only cross-rank operations are a barrier around the timed
region, the maximum of the per-rank times and the sum of the units processed.
"""

from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init(backend: str, device_id: int | None = None) -> None:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT."""
    if dist.is_initialized():
        return
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    kwargs = {}
    if backend == "nccl" and device_id is not None:
        kwargs["device_id"] = torch.device("cuda", device_id)
    dist.init_process_group(backend=backend, **kwargs)


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def combine(elapsed_ms: float, units: float):
    """(max over ranks of elapsed_ms, sum over ranks of units).  Identity without a process group."""
    if not dist.is_initialized():
        return float(elapsed_ms), float(units)
    device = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
