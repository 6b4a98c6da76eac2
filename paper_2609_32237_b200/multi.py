"""Host logic of the multi-GPU bench: one process per GPU, every rank transforms its own
batch (the batched transforms are independent, so there is no data-path collective), and
the timing is the maximum over ranks. Works with any torch.distributed backend (nccl on
GPUs, gloo in the CPU tests)."""
from __future__ import annotations


def max_over_ranks(value: float, device=None) -> float:
    """All-reduce MAX of one float over the default process group (identity if not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(bytes_per_rank: int, ms_per_step_local: float, world: int, device=None):
    """(whole-job GB/s, max-over-ranks ms per step): every rank moved bytes_per_rank per step."""
    ms = max_over_ranks(ms_per_step_local, device)
    return world * bytes_per_rank / (ms * 1e-3) / 1e9, ms


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's own batch (replicas draw different data)."""
    return int(base_seed) + int(rank)
