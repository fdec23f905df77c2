"""Multi-GPU plumbing for the benchmark: one process per GPU, sequences sharded across ranks.

(sequence, v-head) units of the gated delta rule are independent, so the path shards with no
data-path collective: rank r owns a contiguous slice of the global batch and runs the same
kernels on it.  `torch.distributed` is used only to line the ranks up (barrier) and to reduce the
timing (max over ranks).  Works with the "nccl" backend on GPUs and with "gloo" on CPU (tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> None:
    rank, size, _ = world()
    if size > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, rank=rank, world_size=size, **kw)


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def shard(n_global: int, size: int, rank: int) -> range:
    """Contiguous slice of range(n_global) owned by `rank`; slices differ in length by at most 1."""
    base, extra = divmod(n_global, size)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(values, device="cpu") -> list[float]:
    """Element-wise maximum of a short list of floats over all ranks (the slowest rank's times)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_rate(units_per_rank: float, ms_max: float, size: int) -> float:
    """Units per second of the whole job: every rank's units over the slowest rank's time."""
    return size * units_per_rank / (ms_max * 1e-3)
