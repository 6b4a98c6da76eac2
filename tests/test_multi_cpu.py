"""The multi-rank bench logic on CPU: two gloo ranks, each with its own batch and its own
step time; the reported time is the maximum over ranks and the value the whole-job aggregate."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2609_32237_b200 import multi, inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 1.0 + 0.5 * rank                      # rank 1 is the slow one
        gbs, ms = multi.aggregate_throughput(2 << 30, local_ms, world)
        x = inputs.gaussian_complex64((2, 64), multi.rank_seed(1, rank))
        dist.barrier()
        q.put((rank, gbs, ms, float(abs(x).sum())))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_max_time_and_aggregate_value():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, g0, ms0, s0), (r1, g1, ms1, s1) = out
    assert ms0 == ms1 == 1.5                              # the maximum over ranks, on both
    want = 2 * (2 << 30) / 1.5e-3 / 1e9
    assert abs(g0 - want) < 1e-6 and abs(g1 - want) < 1e-6
    assert s0 != s1                                       # each rank drew its own batch


def test_single_process_is_identity():
    from paper_2609_32237_b200 import multi
    gbs, ms = multi.aggregate_throughput(1 << 30, 2.0, 1)
    assert ms == 2.0 and abs(gbs - (1 << 30) / 2e-3 / 1e9) < 1e-9
    assert multi.rank_seed(7, 3) == 10
