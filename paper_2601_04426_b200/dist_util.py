"""Process-group plumbing for the benchmark: one process per GPU, no data-path collective.

Requests are independent, so N GPUs serve N batches side by side (weak scaling).  The only
communication is the barrier around the timed region and the max-over-ranks of the measured time.
"""
from __future__ import annotations

import copy
import os

import torch
import torch.distributed as dist


def world_size() -> int:
    return int(os.environ.get("WORLD_SIZE", "1"))


def init_from_env(backend: str) -> bool:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_* (no-op for one process)."""
    if world_size() <= 1 or dist.is_initialized():
        return dist.is_initialized()
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    dist.init_process_group(backend=backend, rank=int(os.environ["RANK"]), world_size=world_size())
    return True


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rotate_requests(workload, rank: int):
    """Rank r serves the same seeded requests in an order rotated by r (its own batch)."""
    w = copy.copy(workload)
    n = len(w.request_grammar)
    k = (rank * 7) % n if n else 0
    w.request_grammar = w.request_grammar[k:] + w.request_grammar[:k]
    w.trajectories = w.trajectories[k:] + w.trajectories[:k]
    w.documents = w.documents[k:] + w.documents[:k]
    return w


def finish() -> None:
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
