"""Host-side plumbing for running the path on several GPUs of one node.

The path has no exchange step (chunking is per sequence, compression per (layer, sequence, head,
segment), decode per (sequence, head)), so ranks are independent replicas: each owns its own
seeded batch and the only communication is a barrier around the timed region and a MAX over
ranks of the device-side timings.  Works with the ``nccl`` backend (one rank per GPU) and with
``gloo`` on CPU tensors, which is how the logic is tested without GPUs.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def init(backend: str, device: torch.device | None = None) -> None:
    """Join the process group described by MASTER_ADDR / MASTER_PORT / RANK / WORLD_SIZE."""
    if dist.is_initialized():
        return
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)


def rank_workload(w, rank: int):
    """The batch a rank owns: same shape, its own seed (weak scaling: per-GPU work is fixed)."""
    return w if rank == 0 else w.replace(seed=w.seed + 1000 * rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise MAX of a list of floats over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def barrier(device=None) -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if device is not None and torch.device(device).type == "cuda":
        torch.cuda.synchronize(device)


def whole_job_rate(units_per_rank: float, world_size: int, max_ms: float) -> float:
    """Aggregate throughput: units of all ranks over the slowest rank's time."""
    return units_per_rank * world_size / (max_ms * 1e-3)
