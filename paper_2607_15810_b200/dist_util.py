"""Multi-process plumbing of the benchmark: one process per GPU, replicas of the
layer on independent batches (the path has no data-path collective), a barrier,
and the max-over-ranks step time.  Works with NCCL on GPUs and with gloo on CPU
(the latter is what the CPU tests exercise)."""
import os

import torch
import torch.distributed as dist


def env_world():
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend, device=None):
    world, rank, _ = env_world()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    return world, rank


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value, device="cpu"):
    """Largest `value` over all ranks (the slowest rank decides the step time)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world, units_per_rank, ms_per_step):
    """Units all ranks processed per second when each rank does `units_per_rank`
    per step and the step takes `ms_per_step` (max over ranks)."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def shutdown():
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
