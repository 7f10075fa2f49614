"""Multi-GPU plumbing for replicas of the decode path: no collective touches the data path.

Sequences (and heads) are independent in decode attention, so N GPUs each take a batch shard and
run the same single-GPU step.  The only cross-rank traffic is for timing: a barrier and the
max / sum of two scalars.  Backend "nccl" on GPUs, "gloo" in CPU tests.
"""
import torch
import torch.distributed as dist


def init(backend: str, device=None):
    """Initialise the default process group from the torchrun environment (RANK, WORLD_SIZE, ...)."""
    if dist.is_initialized():
        return
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)


def world():
    return dist.get_world_size() if dist.is_initialized() else 1


def rank():
    return dist.get_rank() if dist.is_initialized() else 0


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, ms_this_rank: float, device="cpu") -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    total = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(ms_this_rank, device)
    return total / (ms * 1e-3)
