"""Multi-process plumbing for `bench.py --gpus N`.

The path does not shard: every (batch, head) slab is independent and the method has no
exchange step, so N GPUs run N independent replicas with no data-path collective.  The only
communication is the benchmark's own barrier and the max-over-ranks of the device time."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world():
    """(rank, local_rank, world_size) from the torchrun environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None) -> None:
    rank, _, ws = world()
    if ws > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"),
                                rank=rank, world_size=ws)


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device=None):
    """Whole-job numbers from per-rank ones: time = max over ranks, units = sum over ranks."""
    if not dist.is_initialized():
        return elapsed_ms, units
    dev = device if device is not None else ("cuda" if dist.get_backend() == "nccl" else "cpu")
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
