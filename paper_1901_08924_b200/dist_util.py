"""Process-group plumbing for running independent replicas on several GPUs of one node.

The path has no cross-device exchange (communication is counted, never sent), so ranks only meet
to line up their timed regions and to combine their timings: a barrier, a max and a sum.
"""
import os

import torch
import torch.distributed as dist


def world():
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


def init(backend):
    """Joins the process group described by the torchrun environment (no-op for one process)."""
    size, rank, _ = world()
    if size > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=size)
    return size, rank


def barrier():
    if dist.is_initialized():
        dist.barrier()


def _reduce(value, op, device):
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value, device="cpu"):
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value, device="cpu"):
    return _reduce(value, dist.ReduceOp.SUM, device)


def whole_job_throughput(units_this_rank, ms_this_rank, device="cpu"):
    """Units processed by all ranks divided by the slowest rank's time (units per second)."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
