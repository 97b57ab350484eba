"""Multi-GPU host logic: the path shards over independent (batch, head) units with no data-path
collective - every rank runs its own batch of the same shape (weak scaling) - and the only
communication is the host-side agreement on timing (max over ranks) and the total of the units.

One process per GPU (torch.distributed; NCCL on GPUs, gloo in the CPU tests)."""
import torch
import torch.distributed as dist


def max_over_ranks(value, device="cpu"):
    """Every rank gets the maximum of `value` over all ranks (step time = slowest rank)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank, seconds_max):
    """Whole-job throughput: units processed by all ranks divided by the slowest rank's time."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return units_per_rank / seconds_max
    t = torch.tensor([float(units_per_rank)], dtype=torch.float64)
    if dist.get_backend() == "nccl":
        t = t.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item()) / seconds_max
