"""Multi-GPU plumbing of the benchmark: replicas only.

Token batches are independent, so N GPUs run N copies of the per-GPU workload on their own tokens and
nothing crosses between them on the data path.  What ranks do share is the clock: the timed region is
bracketed by a barrier and the step time of the job is the slowest rank's.  These helpers hold that
logic for `bench.py`; they work on any `torch.distributed` backend (NCCL on the GPUs, gloo in the CPU
tests) and do nothing when the world size is 1.
"""
import os

import torch
import torch.distributed as dist


def world_from_env():
    """(rank, world size, local rank) as torchrun exports them; (0, 1, 0) outside torchrun."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend, device=None):
    """Join the process group named by MASTER_ADDR / MASTER_PORT (no-op for a single process)."""
    _, world, _ = world_from_env()
    if world > 1 and not dist.is_initialized():
        kwargs = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, **kwargs)
    return world


def barrier(device_sync=None):
    """All ranks reach this point, and (device_sync) each rank's queued device work has finished."""
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if device_sync is not None:
        device_sync()


def max_over_ranks(value, device="cpu"):
    """The largest `value` (a float, e.g. milliseconds of the timed region) over all ranks."""
    if not (dist.is_initialized() and dist.get_world_size() > 1):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base_seed, rank):
    """Seed of a rank's own token batch: ranks must not repeat each other's tokens."""
    return base_seed + 100 * rank


def whole_job_rate(units_per_rank, slowest_seconds, world):
    """Aggregate throughput: every rank processed `units_per_rank` in at most `slowest_seconds`."""
    return world * units_per_rank / slowest_seconds


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
