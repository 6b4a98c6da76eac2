"""GPU parity of the range-Doppler chain against the float64 oracle: each
pass on its own, the whole image (relative L2 <= 1e-5 with fp32
intermediates, <= 5e-3 with fp16), and every target's peak cell exactly."""
import numpy as np
import pytest

import oracle
from oracle import quality
from paper_2609_32237_b200 import inputs
from gpu_util import have_gpu, rel_l2, to_device_c64, half_to_c128

pytestmark = pytest.mark.gpu
C64, C32H = 0, 1


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not have_gpu():
        pytest.skip("no CUDA device")


def _gpu_chain(scene, raw, dtype, steps=False, fused=None, layout=None, tile_columns=None):
    """Run the chain through the C ABI. layout: 0 = row-major intermediates and direct column
    kernels (the default), 1 = slab layout, 2 = row-major with every azimuth transform done as
    transpose, row transforms, transpose (the paper's four-pass form); tile_columns: range bins per
    column tile on the slab layout."""
    import torch
    from paper_2609_32237_b200 import binding as B
    p = B.sar_rda_params_create(B.sar_desc_from_scene(scene, dtype))
    try:
        if layout is not None:
            B.sar_rda_set_option(p, "layout", int(layout))
        if tile_columns is not None:
            B.sar_rda_set_option(p, "tile_columns", int(tile_columns))
        if fused is not None:
            B.sar_rda_set_option(p, "fused_rcmc", int(fused))
        need = B.sar_rda_workspace_bytes(p)
        na, nr = scene.n_azimuth, scene.n_range
        image = na * nr * (8 if dtype == C64 else 4)
        assert need == 2 * image
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        B.sar_rda_set_workspace(p, ws.data_ptr(), need)
        rd = to_device_c64(raw)
        out = torch.zeros_like(rd)
        st = torch.cuda.current_stream().cuda_stream
        slab = layout == 1

        def ws_as_complex():
            """The first intermediate image as a row-major complex128 matrix (undoing the slab
            layout: granules of 32 bytes, element (k, n) at ((n // G) * na + k) * G + n % G)."""
            first = ws[:image]
            if dtype == C64:
                a = first.view(torch.complex64).cpu().numpy().astype(np.complex128)
                g = 4
            else:
                a = half_to_c128(first.view(torch.float16).reshape(-1, 2))
                g = 8
            if slab:
                return a.reshape(nr // g, na, g).transpose(1, 0, 2).reshape(na, nr)
            return a.reshape(na, nr)

        if steps:
            inter = []
            for s in range(3):
                B.sar_rda_run_step(rd.data_ptr(), p, out.data_ptr(), s, st)
                torch.cuda.synchronize()
                if s < 2:
                    inter.append(ws_as_complex())
            return out.cpu().numpy(), inter
        B.sar_rda_form_image(rd.data_ptr(), p, out.data_ptr(), st)
        torch.cuda.synchronize()
        return out.cpu().numpy()
    finally:
        B.sar_rda_params_destroy(p)


@pytest.fixture(scope="module")
def small_scene():
    """1024 pulses x 2048 range samples; a 3 m antenna keeps the aperture (about
    520 pulses) inside the frame. Same radar otherwise; noise at 20 dB."""
    sc = inputs.x_band_scene(n_azimuth=1024, n_range=2048, n_targets=0)
    sc.antenna_m = 3.0
    sc.targets = inputs.seeded_target_cells(sc, 5, seed=9)
    raw = inputs.simulate_raw(sc, seed=9)
    p = oracle.sar_params(sc)
    rc = oracle.sar_range_compress(p, raw)
    S = oracle.sar_azimuth_fft(p, rc)
    img = oracle.sar_azimuth_ifft(p, oracle.sar_azimuth_filter(p, oracle.sar_rcmc(p, S)))
    return sc, raw, rc, S, img


LAYOUTS = [(0, None), (1, 2), (1, 4), (2, None)]          # (layout, tile_columns); layout 2: transposes + row transforms


@pytest.mark.parametrize("layout,tile_columns", LAYOUTS)
def test_small_scene_each_pass_fp32(small_scene, layout, tile_columns):
    sc, raw, rc, S, img = small_scene
    got, inter = _gpu_chain(sc, raw, C64, steps=True, layout=layout, tile_columns=tile_columns)
    assert rel_l2(inter[0], rc) <= 1e-5                      # fused range compression
    assert rel_l2(inter[1], S / sc.n_azimuth) <= 1e-5        # azimuth FFT, scaled 1/N_a
    assert rel_l2(got, img) <= 1e-5
    for cell in sc.targets:
        assert quality.peak_cell(got, tuple(cell)) == tuple(cell)


@pytest.mark.parametrize("layout,tile_columns", LAYOUTS)
def test_small_scene_fp16_intermediates(small_scene, layout, tile_columns):
    sc, raw, rc, S, img = small_scene
    got, inter = _gpu_chain(sc, raw, C32H, steps=True, layout=layout, tile_columns=tile_columns)
    assert rel_l2(inter[0], rc) <= 5e-3
    assert rel_l2(inter[1], S / sc.n_azimuth) <= 5e-3
    assert rel_l2(got, img) <= 5e-3
    for cell in sc.targets:
        assert quality.peak_cell(got, tuple(cell)) == tuple(cell)


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("dtype,tol", [(C64, 1e-5), (C32H, 5e-3)])
def test_small_scene_fused_and_unfused_step2_agree(small_scene, dtype, tol, layout):
    """Step 2 as one fused kernel and as row pass + column pass: both within tolerance of the
    oracle, and equal to each other to rounding (with fp16 intermediates the slab layout's row
    pass rounds once more to fp16, which the fused kernel does not)."""
    sc, raw, rc, S, img = small_scene
    a = _gpu_chain(sc, raw, dtype, fused=True, layout=layout)
    b = _gpu_chain(sc, raw, dtype, fused=False, layout=layout)
    assert rel_l2(a, img) <= tol and rel_l2(b, img) <= tol
    assert rel_l2(a, b) <= (2e-6 if (dtype == C64 or layout == 0) else 1e-3)
    for cell in sc.targets:
        assert quality.peak_cell(a, tuple(cell)) == tuple(cell)
        assert quality.peak_cell(b, tuple(cell)) == tuple(cell)


def test_form_image_from_host_buffers(small_scene):
    """sar_rda_form_image_host: raw data in pinned host memory, image back to pinned host memory,
    copies and the chain ordered on one stream; same image as the device-resident call, bit for bit."""
    import torch
    from paper_2609_32237_b200 import binding as B
    sc, raw, rc, S, img = small_scene
    want = _gpu_chain(sc, raw, C64)
    p = B.sar_rda_params_create(B.sar_desc_from_scene(sc, C64))
    try:
        need = B.sar_rda_workspace_bytes(p)
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        B.sar_rda_set_workspace(p, ws.data_ptr(), need)
        h_raw = torch.from_numpy(np.ascontiguousarray(raw, dtype=np.complex64)).pin_memory()
        h_out = torch.zeros_like(h_raw).pin_memory()
        d_raw = torch.zeros(raw.shape, dtype=torch.complex64, device="cuda")
        d_out = torch.zeros_like(d_raw)
        st = torch.cuda.current_stream().cuda_stream
        B.sar_rda_form_image_host(h_raw.data_ptr(), p, h_out.data_ptr(), d_raw.data_ptr(), d_out.data_ptr(), st)
        torch.cuda.synchronize()
        got = h_out.numpy()
        assert rel_l2(got, img) <= 1e-5
        assert np.array_equal(got.view(np.uint64), want.view(np.uint64))
        assert np.array_equal(d_raw.cpu().numpy(), raw.astype(np.complex64))
        with pytest.raises(B.B200FftError) as e:               # null host pointer
            B.sar_rda_form_image_host(0, p, h_out.data_ptr(), d_raw.data_ptr(), d_out.data_ptr(), st)
        assert e.value.status == 1
    finally:
        B.sar_rda_params_destroy(p)


def test_single_on_grid_echo_compresses_to_the_pulse_length():
    sc = inputs.x_band_scene(n_azimuth=1024, n_range=2048, n_targets=0)
    sc.noise_variance = 0.0
    raw = np.zeros((1024, 2048), dtype=np.complex64)
    i = np.arange(-600, 600)
    kappa = sc.chirp_rate / sc.fs_hz ** 2
    raw[5, 900 + i] = np.exp(1j * np.pi * kappa * i.astype(np.float64) ** 2)
    got, inter = _gpu_chain(sc, raw, C64, steps=True)
    assert abs(inter[0][5, 900] - 1200) < 1e-2
    assert np.abs(inter[0][6]).max() == 0


@pytest.mark.parametrize("layout,tile_columns", LAYOUTS)
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("dtype,tol", [(C64, 1e-5), (C32H, 5e-3)])
def test_config4_full_scene(dtype, tol, fused, layout, tile_columns, full_scene):
    """4096 x 4096, 16 seeded unit targets, noise at 20 dB: whole image and peak cells,
    for both forms of step 2 and both intermediate layouts."""
    sc, raw, img = full_scene
    if fused and layout == 2:
        pytest.skip("the transposed form has no fused step 2")
    got = _gpu_chain(sc, raw, dtype, fused=fused, layout=layout, tile_columns=tile_columns)
    err = rel_l2(got, img)
    assert err <= tol, err
    for cell in sc.targets:
        cell = tuple(cell)
        assert quality.peak_cell(got, cell) == cell
        assert quality.peak_cell(img, cell) == cell
    # focus quality matches the reference image's
    cell = tuple(sc.targets[0])
    for axis in (0, 1):
        wg, pg, _ = quality.irw_pslr(quality.cut_through(got.astype(np.complex128), cell, axis))
        wo, po, _ = quality.irw_pslr(quality.cut_through(img, cell, axis))
        assert abs(wg - wo) < 0.01 and abs(pg - po) < 0.05


@pytest.fixture(scope="module")
def l_band_case():
    """The paper's worked L-band scene (wavelength 0.24 m, PRF 500 Hz, 8 m antenna, 20 km) on a
    4096 x 2048 frame with noise: the migration correction shifts rows by up to about 190 bins
    at the edge of the Doppler spectrum, so the moving row windows and their zero fill at the
    row ends run with large shifts."""
    sc = inputs.l_band_scene(n_azimuth=4096, n_range=2048, targets=[(2048, 1024), (1500, 800), (2600, 1390)])
    sc.noise_variance = 0.01
    raw = inputs.simulate_raw(sc, seed=12)
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    return sc, raw, img


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("dtype,tol", [(C64, 1e-5), (C32H, 5e-3)])
def test_l_band_scene_with_large_shifts(dtype, tol, fused, layout, l_band_case):
    sc, raw, img = l_band_case
    got = _gpu_chain(sc, raw, dtype, fused=fused, layout=layout)
    err = rel_l2(got, img)
    assert err <= tol, err
    for cell in sc.targets:
        cell = tuple(cell)
        assert quality.peak_cell(got, cell) == cell
        assert quality.peak_cell(img, cell) == cell


@pytest.fixture(scope="module")
def full_scene():
    sc = inputs.x_band_scene(n_azimuth=4096, n_range=4096, n_targets=16, seed=4)
    raw = inputs.simulate_raw(sc, seed=4)
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    return sc, raw, img


def test_wide_swath_frame():
    """1024 pulses x 8192 range samples: the 8192-point range compression kernel and 128 chunks of the row
    pass, both intermediate types, row-major and slab layouts."""
    sc = inputs.x_band_scene(n_azimuth=1024, n_range=8192, n_targets=0)
    sc.antenna_m = 3.0
    sc.targets = inputs.seeded_target_cells(sc, 4, seed=21)
    raw = inputs.simulate_raw(sc, seed=21)
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    for dtype, tol in ((C64, 1e-5), (C32H, 5e-3)):
        for layout in (0, 1):
            got = _gpu_chain(sc, raw, dtype, layout=layout)
            assert rel_l2(got, img) <= tol
            for cell in sc.targets:
                assert quality.peak_cell(got, tuple(cell)) == tuple(cell)


def test_other_frame_sizes_and_error_paths():
    """A 2048 x 1024 frame with a 5 us pulse (other kernel instantiations), both intermediate
    types and both forms of step 2; then the host-side error paths of the SAR calls."""
    import torch
    from paper_2609_32237_b200 import binding as B
    sc = inputs.x_band_scene(n_azimuth=2048, n_range=1024, n_targets=0)
    sc.antenna_m = 1.5
    sc.pulse_s = 5e-6
    sc.targets = inputs.seeded_target_cells(sc, 3, seed=11)
    raw = inputs.simulate_raw(sc, seed=11)
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    for dtype, tol in ((C64, 1e-5), (C32H, 5e-3)):
        for fused, layout in ((False, 0), (True, 0), (False, 1), (True, 1)):
            got = _gpu_chain(sc, raw, dtype, fused=fused, layout=layout)
            assert rel_l2(got, img) <= tol
            for cell in sc.targets:
                assert quality.peak_cell(got, tuple(cell)) == tuple(cell)
    p = B.sar_rda_params_create(B.sar_desc_from_scene(sc, C64))
    try:
        rd = to_device_c64(raw)
        out = torch.zeros_like(rd)
        with pytest.raises(B.B200FftError) as e:               # no workspace yet
            B.sar_rda_form_image(rd.data_ptr(), p, out.data_ptr(), 0)
        assert e.value.status == 6
        need = B.sar_rda_workspace_bytes(p)
        small = torch.zeros(need // 2, dtype=torch.uint8, device="cuda")   # one image instead of two
        with pytest.raises(B.B200FftError) as e:
            B.sar_rda_set_workspace(p, small.data_ptr(), need // 2)
        assert e.value.status == 6
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        B.sar_rda_set_workspace(p, ws.data_ptr(), need)
        with pytest.raises(B.B200FftError) as e:               # output must not alias the input
            B.sar_rda_form_image(rd.data_ptr(), p, rd.data_ptr(), 0)
        assert e.value.status == 1
        with pytest.raises(B.B200FftError) as e:
            B.sar_rda_set_option(p, "no_such_option", 1)
        assert e.value.status == 1
        with pytest.raises(B.B200FftError) as e:
            B.sar_rda_run_step(rd.data_ptr(), p, out.data_ptr(), 7, 0)
        assert e.value.status == 1
    finally:
        B.sar_rda_params_destroy(p)
    bad = B.sar_desc_from_scene(sc, C64)
    bad.n_azimuth = 512                                          # not a compiled azimuth size
    with pytest.raises(B.B200FftError) as e:
        B.sar_rda_params_create(bad)
    assert e.value.status == 2


def _noise_frame(n_azimuth, n_range, seed):
    g = np.random.default_rng(seed)
    return (g.standard_normal((n_azimuth, n_range)) + 1j * g.standard_normal((n_azimuth, n_range))).astype(np.complex64)


@pytest.mark.parametrize("prf_hz,row_pass", [(1059.0, True), (1060.0, False), (1660.0, False)])
def test_shift_growth_at_the_edge_of_the_row_pass_guard(prf_hz, row_pass):
    """The row pass of step 2 stages 2048 + 128 range samples per CTA and is offered only while the
    integer shift grows by at most 112 bins over 2048 range bins at the Doppler edge. With a 0.24 m
    wavelength at 200 m/s that growth is 111.9 bins at PRF 1059 Hz (accepted; shifts reach ~900 bins)
    and 112.1 at 1060 Hz (refused: step 2 falls back to the fused column kernel); 1660 Hz sits just
    below the largest PRF the calls accept at all (shifts beyond the swath width). White noise as
    the raw frame makes every output pixel depend on the window it was read from."""
    from paper_2609_32237_b200 import binding as B
    sc = inputs.l_band_scene(n_azimuth=1024, n_range=2048, targets=[])
    sc.prf_hz = prf_hz
    raw = _noise_frame(1024, 2048, seed=int(prf_hz))
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    assert np.abs(img).max() > 0
    p = B.sar_rda_params_create(B.sar_desc_from_scene(sc, C64))
    try:
        if row_pass:
            B.sar_rda_set_option(p, "fused_rcmc", 0)
        else:
            with pytest.raises(B.B200FftError) as e:
                B.sar_rda_set_option(p, "fused_rcmc", 0)
            assert e.value.status == 2
    finally:
        B.sar_rda_params_destroy(p)
    for dtype, tol in ((C64, 1e-5), (C32H, 5e-3)):
        assert rel_l2(_gpu_chain(sc, raw, dtype), img) <= tol                   # the default form
        assert rel_l2(_gpu_chain(sc, raw, dtype, fused=True), img) <= tol


@pytest.mark.parametrize("prf_hz,accepted", [(410.0, True), (415.0, False)])
def test_shift_spread_at_the_edge_of_the_slab_guard(prf_hz, accepted):
    """The slab-layout row pass holds 32 Doppler bins x 64 range bins per CTA and is offered only
    while the integer shift spreads by at most 16 bins inside one CTA: 15.9 at PRF 410 Hz, 16.3 at
    415 Hz for this 1024 x 2048 frame."""
    from paper_2609_32237_b200 import binding as B
    sc = inputs.l_band_scene(n_azimuth=1024, n_range=2048, targets=[])
    sc.prf_hz = prf_hz
    raw = _noise_frame(1024, 2048, seed=int(prf_hz))
    if not accepted:
        p = B.sar_rda_params_create(B.sar_desc_from_scene(sc, C64))
        try:
            with pytest.raises(B.B200FftError) as e:
                B.sar_rda_set_option(p, "layout", 1)
            assert e.value.status == 2
        finally:
            B.sar_rda_params_destroy(p)
        return
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    for dtype, tol in ((C64, 1e-5), (C32H, 5e-3)):
        for tile_columns in (2, 4):
            assert rel_l2(_gpu_chain(sc, raw, dtype, layout=1, tile_columns=tile_columns), img) <= tol


def _gpu_sharded(scene, raw, dtype, world):
    """The column-strip decomposition with all `world` ranks on one device: every rank's step 1 (range
    compression scattered into every rank's strip buffer), then every rank's step 2 on its own strip."""
    import torch
    from paper_2609_32237_b200 import binding as B
    desc = B.sar_desc_from_scene(scene, dtype)
    shards = [B.sar_rda_shard_create(desc, r, world) for r in range(world)]
    try:
        geo = [B.sar_rda_shard_get_geometry(s) for s in shards]
        for r, g in enumerate(geo):
            h = B.sar_rda_shard_geometry_of(desc, r, world)
            assert all(getattr(h, f) == getattr(g, f) for f, _ in B.SarShardGeometry._fields_)
        # poisoned workspaces: whatever the kernels do not write shows up in the result
        ws = [torch.full((g.workspace_bytes,), 0x7f, dtype=torch.uint8, device="cuda") for g in geo]
        for s, w, g in zip(shards, ws, geo):
            B.sar_rda_shard_set_workspace(s, w.data_ptr(), g.workspace_bytes)
        rd = to_device_c64(raw)
        ptrs = [w.data_ptr() for w in ws]
        for r, (s, g) in enumerate(zip(shards, geo)):
            rows = rd[g.first_pulse:g.first_pulse + g.pulses]
            assert rows.is_contiguous()
            B.sar_rda_shard_range_compress(s, rows.data_ptr(), ptrs, 0)
        torch.cuda.synchronize()              # every rank's step 1 before any rank's step 2
        image = np.zeros((scene.n_azimuth, scene.n_range), np.complex64)
        for s, g in zip(shards, geo):
            strip = torch.zeros(scene.n_azimuth, g.bins, 2, device="cuda")
            B.sar_rda_shard_azimuth(s, strip.data_ptr(), 0)
            torch.cuda.synchronize()
            image[:, g.first_bin:g.first_bin + g.bins] = strip.cpu().numpy().view(np.complex64)[..., 0]
        return image
    finally:
        for s in shards:
            B.sar_rda_shard_destroy(s)


@pytest.mark.parametrize("world", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,tol", [(C64, 1e-5), (C32H, 5e-3)])
def test_column_strip_decomposition_small_scene(small_scene, world, dtype, tol):
    """Every rank count the decomposition accepts, all ranks emulated on one device: the assembled image against
    the oracle and against the single-device chain; every target's peak cell."""
    sc, raw, _, _, img = small_scene
    got = _gpu_sharded(sc, raw, dtype, world)
    assert rel_l2(got, img) <= tol
    assert rel_l2(got, _gpu_chain(sc, raw, dtype)) <= (2e-6 if dtype == C64 else tol)
    for cell in sc.targets:
        assert quality.peak_cell(got, tuple(cell)) == tuple(cell)


@pytest.mark.parametrize("world", [2, 8])
def test_column_strip_decomposition_large_shifts(world, l_band_case):
    """The L-band scene: the halo on the far side of every strip is about 200 bins wide."""
    from paper_2609_32237_b200 import binding as B
    sc, raw, img = l_band_case
    g = B.sar_rda_shard_geometry_of(B.sar_desc_from_scene(sc, C64), 0, world)
    assert g.halo_right >= 190 and g.halo_left == 8 and g.bins == sc.n_range // world
    got = _gpu_sharded(sc, raw, C64, world)
    assert rel_l2(got, img) <= 1e-5


def test_column_strip_decomposition_refusals():
    from paper_2609_32237_b200 import binding as B
    sc = inputs.l_band_scene(n_azimuth=1024, n_range=1024, targets=[])
    desc = B.sar_desc_from_scene(sc, C64)
    for rank, world, status in ((0, 3, 1), (2, 2, 1), (-1, 2, 1), (0, 8, 2)):     # 8 strips of 128 bins: halos do not fit
        with pytest.raises(B.B200FftError) as e:
            B.sar_rda_shard_geometry_of(desc, rank, world)
        assert e.value.status == status


def test_strip_rank_on_a_process_group_of_one(small_scene):
    """The launcher for real devices (symmetric-memory strip buffers, barrier between the steps) with a
    process group of one rank: both barrier styles, against the oracle."""
    import os
    import socket
    import torch
    import torch.distributed as dist
    from paper_2609_32237_b200 import binding as B, multi
    sc, raw, _, _, img = small_scene
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        rd = to_device_c64(raw)
        for host_barrier in (True, False):
            job = multi.SarStripRank(B.sar_desc_from_scene(sc, C64), host_barrier=host_barrier)
            try:
                assert job.geometry.pulses == sc.n_azimuth and job.geometry.bins == sc.n_range
                out = job.form(rd)
                torch.cuda.synchronize()
                got = out.cpu().numpy().view(np.complex64)[..., 0]
                assert rel_l2(got, img) <= 1e-5
            finally:
                job.close()
    finally:
        dist.destroy_process_group()
