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


def _strip_worker(rank, world, port, q):
    """One rank of the column-strip image formation on CPU: the library supplies the geometry (host
    arithmetic), the oracle does the arithmetic, gloo carries the exchange."""
    sys.path.insert(0, ROOT)
    import copy
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2609_32237_b200 import binding as B, inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        sc = inputs.l_band_scene(n_azimuth=512, n_range=1024, targets=[])
        g0 = np.random.default_rng(5)
        raw = (g0.standard_normal((512, 1024)) + 1j * g0.standard_normal((512, 1024))).astype(np.complex64)
        geo = [B.sar_rda_shard_geometry_of(B.sar_desc_from_scene(sc, 0), r, world) for r in range(world)]
        me = geo[rank]
        p = oracle.sar_params(sc)
        # step 1: this rank's pulses, whole range lines (the other rows stay zero and are not used)
        mine = np.zeros((sc.n_azimuth, sc.n_range), np.complex128)
        mine[me.first_pulse:me.first_pulse + me.pulses] = raw[me.first_pulse:me.first_pulse + me.pulses]
        rc = oracle.sar_range_compress(p, mine)[me.first_pulse:me.first_pulse + me.pulses]
        # exchange: every rank ends up with all pulses of its strip and halos
        blocks = [torch.zeros(geo[r].pulses, sc.n_range, dtype=torch.complex128) for r in range(world)]
        dist.all_gather(blocks, torch.from_numpy(np.ascontiguousarray(rc)))
        full = np.concatenate([b.numpy() for b in blocks], axis=0)
        first = me.first_bin - me.halo_left                  # bin of the whole frame at column 0 of the strip
        strip = np.zeros((sc.n_azimuth, me.strip_width), np.complex128)
        lo, hi = max(first, 0), min(first + me.strip_width, sc.n_range)
        strip[:, lo - first:hi - first] = full[:, lo:hi]      # bins outside the frame stay zero
        # step 2 on the strip as a frame of its own
        ss = copy.copy(sc)
        ss.n_range = int(me.strip_width)
        ss.r_center_m = sc.r_center_m + (first + me.strip_width // 2 - sc.n_range // 2) * sc.range_bin_m
        ps = oracle.sar_params(ss)
        S = oracle.sar_azimuth_fft(ps, strip)
        img = oracle.sar_azimuth_ifft(ps, oracle.sar_azimuth_filter(ps, oracle.sar_rcmc(ps, S)))
        keep = np.ascontiguousarray(img[:, me.halo_left:me.halo_left + me.bins])
        parts = [torch.zeros(sc.n_azimuth, geo[r].bins, dtype=torch.complex128) for r in range(world)]
        dist.all_gather(parts, torch.from_numpy(keep))
        if rank == 0:
            whole = np.concatenate([t.numpy() for t in parts], axis=1)
            want = oracle.sar_rda(p, raw)
            err = float(np.linalg.norm(whole - want) / np.linalg.norm(want))
            q.put((err, int(me.halo_right), int(me.strip_width)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_form_an_image_by_column_strips():
    """The decomposition of sar_rda_shard_* with the oracle as the arithmetic: pulses split for range
    compression, range bins split (with the library's halos) for the azimuth steps; the assembled image
    equals the undivided oracle image to float64 rounding, which it only does if the halos cover the
    interpolator's reach (about 190 bins of migration in this scene)."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_strip_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    err, halo_right, width = q.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert halo_right >= 190 and width == 8 + 512 + halo_right
    assert err <= 1e-11


def test_strip_halos_cover_the_largest_migration_the_oracle_computes():
    """halo_right of sar_rda_shard_geometry_of against the oracle's migration (in range bins) at the far
    edge of the swath over every Doppler bin: the interpolator reads up to floor(migration) + 4 bins ahead."""
    import math
    import oracle
    from paper_2609_32237_b200 import binding as B, inputs
    for sc in (inputs.x_band_scene(n_azimuth=1024, n_range=2048, n_targets=0),
               inputs.l_band_scene(n_azimuth=1024, n_range=2048, targets=[])):
        p = oracle.sar_params(sc)
        worst = max(oracle.sar_migration_bins(p, k, sc.n_range - 1) for k in range(sc.n_azimuth))
        least = min(oracle.sar_migration_bins(p, k, 0) for k in range(sc.n_azimuth))
        assert least >= 0.0                                   # the window never reaches further back than 3 bins
        for world in (1, 2, 4):
            g = B.sar_rda_shard_geometry_of(B.sar_desc_from_scene(sc, 0), world - 1, world)
            assert g.halo_left >= 3
            assert g.halo_right >= math.floor(worst) + 4
            assert g.halo_right <= math.floor(worst) + 4 + 9  # rounded up to a multiple of 8, one bin of slack
            assert g.halo_right % 8 == 0 and g.strip_width == g.halo_left + g.bins + g.halo_right
