"""Multi-process plumbing for replica runs: the composed forward has no exchange step (every
workload is independent over rows / images / batch elements and weights are replicated), so ranks
only agree on when the timed region starts and on the slowest rank's times.  Works with any
torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device=None):
    """Initialise the default process group if WORLD_SIZE > 1.  Returns True if distributed."""
    _, _, world = env_world()
    if world <= 1:
        return False
    if not dist.is_initialized():
        kw = {}
        if device is not None and backend == "nccl":
            kw["device_id"] = device
        dist.init_process_group(backend, **kw)
    return True


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over all ranks of a list of floats (the job's time is the slowest
    rank's time).  Single-process: returns the values unchanged."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def shard_rows(n_rows: int, rank: int, world: int):
    """Contiguous row range [lo, hi) of rank `rank` when n_rows independent rows are split over
    `world` replicas (strong-scaling use; the benchmark itself runs whole workloads per rank)."""
    base, rem = divmod(n_rows, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def aggregate_throughput(work_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return work_per_rank * world / seconds_max
