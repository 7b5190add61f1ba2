"""Replica bookkeeping for multi-process runs (one process per GPU, no data-path collective): rendezvous, barrier,
and the maximum over ranks of a per-rank time.  The mixer shards over batch rows without any exchange, so this is all
the communication a multi-GPU run has.  Works with backend "nccl" (GPU) and "gloo" (CPU, used by the tests)."""
from __future__ import annotations

import os


def env_ranks():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str, local_rank: int = 0):
    """Joins the process group when WORLD_SIZE > 1 (rendezvous on 127.0.0.1 unless MASTER_ADDR is set)."""
    import torch
    import torch.distributed as dist
    _, _, world = env_ranks()
    if world <= 1 or dist.is_initialized():
        return
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        dist.init_process_group(backend)
    dist.barrier()


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The slowest rank's time: what a whole-job throughput has to be divided by."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, steps: int, ms_total_max: float) -> float:
    """Units all ranks processed per second: every rank does the same work (weak scaling), the slowest one sets the time."""
    _, _, world = env_ranks()
    return world * units_per_rank * steps / (ms_total_max * 1e-3)


def shutdown():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
