"""Multi-process plumbing of the benchmark: one process per GPU, no data-path collective.

Every image is independent through the whole block, so N ranks run N
independent batches (weak scaling); the only exchange is the reduction of the
measured times (maximum over ranks) that the throughput is computed from.
The helpers work on any torch.distributed backend (nccl on GPUs, gloo on CPU).
"""
import os

import torch
import torch.distributed as dist


def env_world():
    """(world_size, rank, local_rank) from the launcher's environment (1, 0, 0 when absent)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend, local_rank=0):
    """Joins the process group when launched with WORLD_SIZE > 1; returns (world, rank)."""
    world, rank, _ = env_world()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend)
    return world, rank


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over all ranks of a list of floats (identity for one process)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def rank_seed(seed, rank):
    """Every rank draws its own batch: same generator, disjoint seed ranges."""
    return int(seed) + 100000 * int(rank)


def job_throughput(units_per_rank_per_step, steps, world, slowest_ms):
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return world * units_per_rank_per_step * steps / (slowest_ms / 1e3)


def finish():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
