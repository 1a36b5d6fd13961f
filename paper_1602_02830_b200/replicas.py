"""Multi-GPU plumbing of the benchmark: batch rows are independent through every step of the path, so N GPUs
run N independent replicas (one process per GPU, each with its own batch) and no data-path collective exists.
The only communication is the barrier around the timed region and the max-over-ranks of the device times."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world():
    """(world_size, rank, local_rank) from the torchrun environment (1, 0, 0 when launched plainly)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: "torch.device | None" = None) -> None:
    if world()[0] > 1 and not dist.is_initialized():
        if device is not None and backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over all ranks of a list of floats (the slowest rank defines the job's time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(units_per_rank: float, ms_per_step_max: float, world_size: int) -> float:
    """Whole-job units per second when every rank processes `units_per_rank` per step (weak scaling)."""
    return world_size * units_per_rank / (ms_per_step_max / 1e3)


def rank_seed(base_seed: int, rank: int):
    """Seed of rank's own batch: rank 0 keeps the configuration's seed, the others derive theirs from it."""
    return base_seed if rank == 0 else [base_seed, rank]


def finish() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
