"""Process-group plumbing for multi-GPU runs (one process per GPU).

The hot path has no exchange step: sessions (and KV heads) are independent problems, so ranks are given
disjoint sessions and no data-path collective exists.  torch.distributed is used only for the timing
contract: a barrier on both sides of the timed region and the maximum of the per-rank times.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as td


def init_from_env(n_gpus: int, backend: str = "nccl"):
    """Returns (rank, world, local_rank).  With WORLD_SIZE > 1 in the environment (torchrun) the process
    group is created; a single process needs none."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not td.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        kw = {}
        if backend == "nccl":
            kw["device_id"] = torch.device("cuda", local_rank)
        td.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    if world != max(n_gpus, 1) and rank == 0 and world > 1:
        raise SystemExit(f"--gpus {n_gpus} does not match WORLD_SIZE {world}")
    return rank, world, local_rank


def sessions_of_rank(rank: int, world: int, n_sessions: int):
    """Round-robin assignment of independent sessions to ranks; every session goes to exactly one rank."""
    return [s for s in range(n_sessions) if s % world == rank]


def _tensor(x: float):
    if td.get_backend() == "nccl":
        return torch.tensor([x], dtype=torch.float64, device=torch.device("cuda", torch.cuda.current_device()))
    return torch.tensor([x], dtype=torch.float64)


def barrier():
    if td.is_available() and td.is_initialized():
        td.barrier()


def max_over_ranks(x: float) -> float:
    if td.is_available() and td.is_initialized():
        t = _tensor(float(x))
        td.all_reduce(t, op=td.ReduceOp.MAX)
        return float(t.item())
    return float(x)


def sum_over_ranks(x: float) -> float:
    if td.is_available() and td.is_initialized():
        t = _tensor(float(x))
        td.all_reduce(t, op=td.ReduceOp.SUM)
        return float(t.item())
    return float(x)


def shutdown():
    if td.is_available() and td.is_initialized():
        td.destroy_process_group()
