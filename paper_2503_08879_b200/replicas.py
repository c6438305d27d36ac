"""Process-group plumbing for running independent replicas of the path, one per GPU.

The four steps never exchange data between GPUs (layers, batch entries and KV heads are independent),
so the only collectives are the ones a benchmark needs: a barrier around the timed region and a
max / sum over the ranks' measurements.  Backend "nccl" on GPUs, "gloo" for the CPU tests.
"""

from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when not launched by one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str = "nccl", device: torch.device | None = None) -> tuple[int, int]:
    """Join the process group if there is more than one rank.  Returns (rank, world_size)."""
    rank, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def _reduce(value: float, op, device) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
