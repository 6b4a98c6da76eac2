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


class SarStripRank:
    """One rank of the SAR image formation by column strips on real devices: one process per GPU,
    `torch.distributed` initialised (backend nccl), the current CUDA device this rank's.

    The strip buffers live in symmetric memory so that every rank can address every other rank's
    buffer; the exchange itself is the epilogue of the range-compression kernel (plain stores to
    the owners' buffers, every store addressed to one buffer), and the only synchronisation between the two steps is
    a barrier: on the device through the symmetric-memory signal pads (default), or on the host
    (`host_barrier=True`: stream synchronise, then the process group's barrier)."""

    def __init__(self, desc, group=None, host_barrier: bool = False):
        import os
        import torch
        import torch.distributed as dist
        from . import binding as B
        os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")   # peer pointers only
        import torch.distributed._symmetric_memory as symm
        self._B = B
        self.group = group if group is not None else dist.group.WORLD
        self.rank, self.world = dist.get_rank(self.group), dist.get_world_size(self.group)
        self.host_barrier = host_barrier
        self.shard = B.sar_rda_shard_create(desc, self.rank, self.world)
        self.geometry = B.sar_rda_shard_get_geometry(self.shard)
        device = torch.device("cuda", torch.cuda.current_device())
        self.workspace = symm.empty(int(self.geometry.workspace_bytes), dtype=torch.uint8, device=device)
        self.handle = symm.rendezvous(self.workspace, self.group)
        self.strips = [int(p) for p in self.handle.buffer_ptrs]
        if self.strips[self.rank] != self.workspace.data_ptr():
            raise RuntimeError("symmetric memory: this rank's own buffer address does not match")
        B.sar_rda_shard_set_workspace(self.shard, self.workspace.data_ptr(), int(self.geometry.workspace_bytes))
        self.image_strip = torch.empty(int(desc.n_azimuth), int(self.geometry.bins), 2, dtype=torch.float32, device=device)

    def _barrier(self):
        import torch
        import torch.distributed as dist
        if self.host_barrier:
            torch.cuda.current_stream().synchronize()
            dist.barrier(self.group)
        else:
            self.handle.barrier()

    def form(self, raw_rows):
        """raw_rows: this rank's pulses (geometry.pulses x n_range complex64 as a float32 tensor with a
        trailing dimension of 2, contiguous, on this device). Returns this rank's strip of the image
        (n_azimuth x geometry.bins x 2, float32), valid once the current stream has finished."""
        import torch
        stream = torch.cuda.current_stream().cuda_stream
        self._B.sar_rda_shard_range_compress(self.shard, raw_rows.data_ptr(), self.strips, stream)
        self._barrier()          # every rank's rows are in every strip
        self._B.sar_rda_shard_azimuth(self.shard, self.image_strip.data_ptr(), stream)
        self._barrier()          # the strip buffers may be overwritten by the next image
        return self.image_strip

    def close(self):
        if self.shard:
            self._B.sar_rda_shard_destroy(self.shard)
            self.shard = None
