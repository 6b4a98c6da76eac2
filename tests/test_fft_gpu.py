"""GPU parity: the CUDA path, called through the C ABI, against the float64
oracle on the same seeded inputs. Tolerances: relative L2 <= 1e-5 for fp32
storage, <= 5e-3 for fp16 storage (worst single transform and pooled)."""
import numpy as np
import pytest

import oracle
from paper_2609_32237_b200 import inputs
from gpu_util import (have_gpu, rel_l2, worst_rel_l2, to_device_c64, to_device_half, run_fft, half_to_c128)

pytestmark = pytest.mark.gpu

TOL32 = 1e-5
TOL16 = 5e-3


_TIMEOUTS = {}


def _timeouts_at_start(B):
    """Bounded waits that gave up before this test started (the give-up test raises the counter on
    purpose; every other test must leave it where it found it)."""
    return _TIMEOUTS["now"]


@pytest.fixture(autouse=True)
def _note_timeouts():
    if have_gpu():
        from paper_2609_32237_b200 import binding as B
        _TIMEOUTS["now"] = B.tma_timeouts()
    yield


FWD, INV = -1, 1
C64, C32H = 0, 1


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not have_gpu():
        pytest.skip("no CUDA device")


def _check_rows(n, batch, seed, dist=None, gaussian=False, direction=FWD, options=None, tol=TOL32):
    dist = dist or n
    gen = inputs.gaussian_complex64 if gaussian else inputs.uniform_complex64
    buf = gen((batch, dist), seed)
    x = buf[:, :n]
    want = oracle.fft_rows(x.astype(np.complex128), direction)
    got = run_fft(to_device_c64(buf), n, batch, 1, dist, direction, C64, options=options).cpu().numpy()
    worst, pooled = worst_rel_l2(got[:, :n], want)
    assert worst <= tol and pooled <= tol, (n, batch, worst, pooled)
    if dist > n:   # padding between transforms must stay untouched (output buffer was zero-filled)
        assert np.all(got[:, n:] == 0)
    return worst


def test_config0_whole_batch_and_round_trip():
    """N = 1024, batch 256, uniform [-1, 1), seed 0: every transform against the direct DFT."""
    x = inputs.uniform_complex64((256, 1024), 0)
    want = oracle.fft_rows(x.astype(np.complex128), FWD)
    xd = to_device_c64(x)
    y = run_fft(xd, 1024, 256, 1, 1024, FWD, C64)
    worst, pooled = worst_rel_l2(y.cpu().numpy(), want)
    assert worst <= TOL32 and pooled <= TOL32
    back = run_fft(y, 1024, 256, 1, 1024, INV, C64).cpu().numpy()
    assert rel_l2(back, x) <= TOL32
    want_inv = oracle.fft_rows(x.astype(np.complex128), INV)
    got_inv = run_fft(xd, 1024, 256, 1, 1024, INV, C64).cpu().numpy()
    assert max(worst_rel_l2(got_inv, want_inv)) <= TOL32


@pytest.mark.parametrize("n", [256, 512, 1024, 2048, 4096, 8192, 16384])
@pytest.mark.parametrize("direction", [FWD, INV])
def test_rows_every_size_ragged_batch(n, direction):
    # batches that do not fill the last CTA of multi-transform configurations
    for batch in (1, 5, 37):
        _check_rows(n, batch, seed=100 + n % 97 + batch, direction=direction, gaussian=(batch == 37))


def test_rows_with_padding_between_transforms():
    _check_rows(4096, 9, seed=7, dist=4096 + 6)
    _check_rows(1024, 11, seed=8, dist=1024 + 2)


def test_rows_closed_forms_on_gpu():
    n = 8192
    x = np.zeros((3, n), dtype=np.complex64)
    x[0, 0] = 1                                  # impulse -> ones
    x[1, :] = 1                                  # ones -> n * delta
    x[2, :] = np.exp(2j * np.pi * 77 * np.arange(n) / n)   # tone -> n * delta at 77
    y = run_fft(to_device_c64(x), n, 3, 1, n, FWD, C64).cpu().numpy()
    assert np.abs(y[0] - 1).max() < 1e-6
    e = np.zeros(n); e[0] = n
    assert np.abs(y[1] - e).max() < 1e-2
    e = np.zeros(n); e[77] = n
    assert np.abs(y[2] - e).max() < 0.2 and abs(y[2, 77] - n) < 0.05


def test_rows_in_place_and_deterministic():
    x = inputs.gaussian_complex64((6, 4096), 21)
    a = run_fft(to_device_c64(x), 4096, 6, 1, 4096, FWD, C64).cpu().numpy()
    b = run_fft(to_device_c64(x), 4096, 6, 1, 4096, FWD, C64, inplace=True).cpu().numpy()
    c = run_fft(to_device_c64(x), 4096, 6, 1, 4096, FWD, C64).cpu().numpy()
    assert np.array_equal(a.view(np.uint64), b.view(np.uint64))
    assert np.array_equal(a.view(np.uint64), c.view(np.uint64))


@pytest.mark.parametrize("n", [1024, 4096, 8192, 16384])
@pytest.mark.parametrize("direction", [FWD, INV])
def test_rows_fp16_storage(n, direction):
    batch = 6
    x = inputs.gaussian_complex64((batch, n), 2)
    if direction == INV:
        x = x * np.float32(8.0)
    h = inputs.to_half_storage(x)
    want = oracle.fft_rows(inputs.from_half_storage(h), direction)   # oracle sees the fp16-rounded input
    got = half_to_c128(run_fft(to_device_half(h), n, batch, 1, n, direction, C32H))
    worst, pooled = worst_rel_l2(got, want)
    assert worst <= TOL16 and pooled <= TOL16
    assert -20 * np.log10(pooled) > 60.0       # fp32 exchange: well above the gate (paper: ~73.6 dB)


@pytest.mark.parametrize("n,cols,ld", [(256, 8, 8), (512, 12, 16), (1024, 20, 20), (2048, 8, 10),
                                       (4096, 12, 12), (8192, 6, 6)])
@pytest.mark.parametrize("direction", [FWD, INV])
def test_columns(n, cols, ld, direction):
    m = inputs.uniform_complex64((n, ld), 3)
    want = oracle.fft_cols(m[:, :cols].astype(np.complex128), direction)
    got = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64).cpu().numpy()
    assert rel_l2(got[:, :cols], want) <= TOL32
    per_col = np.linalg.norm(got[:, :cols] - want, axis=0) / np.linalg.norm(want, axis=0)
    assert per_col.max() <= TOL32
    if ld > cols:
        assert np.all(got[:, cols:] == 0)


@pytest.mark.parametrize("n,cl", [(8192, 2), (8192, 4), (16384, 2), (16384, 4)])
def test_rows_cluster_variants(n, cl):
    """The same transform with a tile shared by a cluster of 2 or 4 CTAs (first
    exchange through distributed shared memory): whole batch against the oracle."""
    _check_rows(n, 5, seed=90 + cl, options={"cluster": cl})
    _check_rows(n, 3, seed=91 + cl, direction=INV, gaussian=True, options={"cluster": cl})


@pytest.mark.parametrize("n,cols,cl", [(2048, 8, 2), (4096, 12, 2), (4096, 12, 4), (8192, 6, 2)])
def test_columns_cluster_variants(n, cols, cl):
    m = inputs.uniform_complex64((n, cols), 33)
    want = oracle.fft_cols(m.astype(np.complex128), FWD)
    got = run_fft(to_device_c64(m), n, cols, cols, 1, FWD, C64, options={"cluster": cl}).cpu().numpy()
    per_col = np.linalg.norm(got - want, axis=0) / np.linalg.norm(want, axis=0)
    assert per_col.max() <= TOL32


def test_columns_fp16_and_in_place():
    n, cols = 4096, 8
    m = inputs.uniform_complex64((n, cols), 31)
    h = inputs.to_half_storage(m)
    want = oracle.fft_cols(inputs.from_half_storage(h), FWD)
    got = half_to_c128(run_fft(to_device_half(h), n, cols, cols, 1, FWD, C32H, inplace=True))
    assert rel_l2(got, want) <= TOL16


def test_2d_small():
    m = inputs.uniform_complex64((512, 256), 32)
    want = oracle.fft2d(m.astype(np.complex128))
    d = to_device_c64(m)
    d = run_fft(d, 256, 512, 1, 256, FWD, C64, inplace=True)
    d = run_fft(d, 512, 256, 256, 1, FWD, C64, inplace=True)
    assert rel_l2(d.cpu().numpy(), want) <= TOL32


def test_config3_columns_and_2d_full():
    """4096 x 4096 row-major, uniform [-1, 1), seed 3: all columns, then the full 2-D transform."""
    m = inputs.uniform_complex64((4096, 4096), 3)
    want_cols = oracle.fft_cols(m.astype(np.complex128), FWD)
    d = to_device_c64(m)
    got = run_fft(d, 4096, 4096, 4096, 1, FWD, C64).cpu().numpy()
    per_col = np.linalg.norm(got - want_cols, axis=0) / np.linalg.norm(want_cols, axis=0)
    assert per_col.max() <= TOL32 and rel_l2(got, want_cols) <= TOL32
    del want_cols
    want2d = oracle.fft2d(m.astype(np.complex128))
    d = run_fft(d, 4096, 4096, 1, 4096, FWD, C64, inplace=True)
    d = run_fft(d, 4096, 4096, 4096, 1, FWD, C64, inplace=True)
    assert rel_l2(d.cpu().numpy(), want2d) <= TOL32


@pytest.mark.parametrize("n", [4096, 8192, 16384, 32768])
@pytest.mark.parametrize("direction", [FWD, INV])
def test_four_step_forced_at_single_pass_sizes(n, direction):
    """The two-pass split forced at sizes the single-pass kernels also cover
    (the paper's regression-test idea): whole batch against the oracle."""
    _check_rows(n, 5, seed=41, direction=direction, options={"four_step": 1})


@pytest.mark.parametrize("lg", [15, 16, 17, 18, 19, 20])
def test_four_step_large(lg):
    n = 1 << lg
    batch = 3 if lg < 20 else 2
    _check_rows(n, batch, seed=50 + lg, gaussian=True)
    _check_rows(n, batch, seed=60 + lg, direction=INV)


@pytest.mark.parametrize("lg,n1", [(16, 64), (16, 1024), (17, 128), (17, 512), (18, 64), (18, 1024),
                                   (19, 128), (19, 1024), (20, 512), (20, 1024)])
def test_four_step_other_splits(lg, n1):
    """n = n1 * n2 with a requested n1 (option split_n1) instead of the default: every pass-1 length
    64..1024 and every pass-2 length 64..4096 occurs once; a split without kernels is refused."""
    from paper_2609_32237_b200 import binding as B
    n = 1 << lg
    _check_rows(n, 2, seed=80 + lg, gaussian=True, options={"four_step": 1, "split_n1": n1})
    _check_rows(n, 2, seed=90 + lg, direction=INV, options={"four_step": 1, "split_n1": n1})
    if lg == 20:
        plan = B.fft_plan_create(n, 2, 1, n, FWD, C64)
        try:
            for bad in (128, 96, 2048):          # n2 = 8192 has no pass 2; not a power of two; n1 too long
                with pytest.raises(B.B200FftError) as e:
                    B.fft_plan_set_option(plan, "split_n1", bad)
                assert e.value.status == 2
        finally:
            B.fft_plan_destroy(plan)


def test_four_step_fp16_and_workspace_errors():
    import torch
    from paper_2609_32237_b200 import binding as B
    n, batch = 1 << 16, 2
    x = inputs.gaussian_complex64((batch, n), 71)
    h = inputs.to_half_storage(x)
    want = oracle.fft_rows(inputs.from_half_storage(h), FWD)
    got = half_to_c128(run_fft(to_device_half(h), n, batch, 1, n, FWD, C32H))
    assert max(worst_rel_l2(got, want)) <= TOL16
    plan = B.fft_plan_create(n, batch, 1, n, FWD, C64)
    try:
        need = B.fft_plan_workspace_bytes(plan)
        assert need == n * batch * 8
        d = to_device_c64(x)
        with pytest.raises(B.B200FftError) as e:
            B.fft_execute(plan, d.data_ptr(), d.data_ptr(), 0)
        assert e.value.status == 6
        small = torch.empty(need // 2, dtype=torch.uint8, device="cuda")
        with pytest.raises(B.B200FftError) as e:
            B.fft_plan_set_workspace(plan, small.data_ptr(), need // 2)
        assert e.value.status == 6
        with pytest.raises(B.B200FftError) as e:
            B.fft_execute(plan, d.data_ptr() + 8, d.data_ptr(), 0)
        assert e.value.status == 3
    finally:
        B.fft_plan_destroy(plan)


def _sampled_full_size(n, batch, seed, dtype, direction=FWD):
    """Full-size batch in the launch configuration the bench times: 64 sampled
    transforms against the oracle, plus two whole-batch invariants computed
    outside the library (Parseval and the DC bin)."""
    import torch
    x = inputs.gaussian_complex64((batch, n), seed)
    idx = inputs.sample_indices(batch, 64, seed)
    if dtype == C64:
        xd = to_device_c64(x)
        y = run_fft(xd, n, batch, 1, n, direction, C64)
        got = y[torch.from_numpy(idx).cuda()].cpu().numpy()
        want = oracle.fft_rows(x[idx].astype(np.complex128), direction)
        tol = TOL32
        yc, xc = y, xd
    else:
        h = inputs.to_half_storage(x)
        del x
        hd = to_device_half(h)
        y = run_fft(hd, n, batch, 1, n, direction, C32H)
        got = half_to_c128(y[torch.from_numpy(idx).cuda()])
        want = oracle.fft_rows(inputs.from_half_storage(h[idx]), direction)
        tol = TOL16
        yc = torch.view_as_complex(y.float())
        xc = torch.view_as_complex(hd.float())
    worst, pooled = worst_rel_l2(got, want)
    assert worst <= tol and pooled <= tol, (worst, pooled)
    if direction == FWD:
        ex = (xc.abs().double() ** 2).sum(-1)
        ey = (yc.abs().double() ** 2).sum(-1)
        assert float(((ey - n * ex).abs() / (n * ex)).max()) <= (1e-5 if dtype == C64 else 5e-3)
        dc = xc.to(torch.complex128).sum(-1)
        scale = float(n) ** 0.5 * 2.0
        assert float((yc[:, 0].to(torch.complex128) - dc).abs().max()) <= (1e-4 if dtype == C64 else 0.2) * scale
    return pooled


def test_config1_full_size_forward_and_inverse():
    """N = 4096, batch 32768 (1 GiB), Gaussian sigma = 1, seed 1."""
    _sampled_full_size(4096, 32768, 1, C64, FWD)
    _sampled_full_size(4096, 32768, 1, C64, INV)


@pytest.mark.parametrize("n,batch", [(8192, 16384), (16384, 8192)])
@pytest.mark.parametrize("dtype", [C64, C32H])
def test_config2_full_size(n, batch, dtype):
    """N = 8192 x 16384 and N = 16384 x 8192, Gaussian, seed 2, fp32 and fp16 storage."""
    _sampled_full_size(n, batch, 2, dtype, FWD)



def test_table_twiddles_variant_matches():
    """First-stage twiddles all loaded from the table (test knob) against the default,
    which loads one row and forms the other powers by multiplication."""
    x = inputs.gaussian_complex64((6, 4096), 96)
    want = oracle.fft_rows(x.astype(np.complex128), FWD)
    a = run_fft(to_device_c64(x), 4096, 6, 1, 4096, FWD, C64).cpu().numpy()
    b = run_fft(to_device_c64(x), 4096, 6, 1, 4096, FWD, C64, options={"alt_factorisation": 1}).cpu().numpy()
    assert max(worst_rel_l2(a, want)) <= TOL32 and max(worst_rel_l2(b, want)) <= TOL32
    assert rel_l2(a, b) <= 1e-6
    # the four-stage factorisation of 16384 (16 x 4 x 16 x 16) against the default 32 x 32 x 16
    x = inputs.gaussian_complex64((3, 16384), 94)
    want = oracle.fft_rows(x.astype(np.complex128), INV)
    a = run_fft(to_device_c64(x), 16384, 3, 1, 16384, INV, C64).cpu().numpy()
    b = run_fft(to_device_c64(x), 16384, 3, 1, 16384, INV, C64, options={"alt_factorisation": 1}).cpu().numpy()
    assert max(worst_rel_l2(a, want)) <= TOL32 and max(worst_rel_l2(b, want)) <= TOL32


@pytest.mark.parametrize("n,cols,ld,dtype", [(2048, 16, 24, C64), (4096, 16, 24, C64), (4096, 1236, 1240, C64),
                                             (4096, 16, 24, C32H), (4096, 1236, 1240, C32H)])
def test_columns_streaming_kernel(n, cols, ld, dtype, kind=1):
    """The persistent column kernel whose tiles arrive and leave through the tensor memory
    accelerator (plan option "stream"; the default for large 4096-row matrices): sampled columns
    against the oracle, everything against the plain-load kernel, padding untouched, in place,
    and no bounded wait ran out. 1236 columns are 309 tiles: two full rounds over 148 CTAs and a
    ragged third."""
    from paper_2609_32237_b200 import binding as B
    m = inputs.uniform_complex64((n, ld), 36)
    tol = TOL32 if dtype == C64 else TOL16
    pick = sorted(set([0, 1, 2, 3, cols - 4, cols - 1] + list(range(5, cols, max(1, cols // 24)))))
    for direction in (FWD, INV):
        if dtype == C64:
            dev = to_device_c64(m)
            src = m.astype(np.complex128)
        else:
            h = inputs.to_half_storage(m)
            dev = to_device_half(h)
            src = inputs.from_half_storage(h)
        want = oracle.fft_cols(src[:, pick], direction)
        got_t = run_fft(dev, n, cols, ld, 1, direction, dtype, options={"stream": kind})
        plain_t = run_fft(dev, n, cols, ld, 1, direction, dtype, options={"stream": 0, "cluster": 1})
        if dtype == C64:
            got, plain = got_t.cpu().numpy(), plain_t.cpu().numpy()
        else:
            got, plain = half_to_c128(got_t), half_to_c128(plain_t)
        per_col = np.linalg.norm(got[:, pick] - want, axis=0) / np.linalg.norm(want, axis=0)
        assert per_col.max() <= tol
        assert rel_l2(got[:, :cols], plain[:, :cols]) <= (2e-7 if dtype == C64 else 2e-4)
        assert np.all(got[:, cols:] == 0)
        inplace = run_fft(dev.clone(), n, cols, ld, 1, direction, dtype, inplace=True, options={"stream": kind})
        assert bool((inplace[:, :cols] == got_t[:, :cols]).all())
    assert B.tma_timeouts() == _timeouts_at_start(B)


def test_bounded_wait_gives_up_and_the_gpu_stays_usable(kind=1):
    """The streaming kernel's wait for its copies is bounded. With the test knob "starve_wait" the
    consumer polls a barrier that nothing ever completes (the copies themselves are counted on
    another one and do land), and with "wait_polls" the limit is 1024 polls: every CTA gives up
    once, waits for its copies in flight and returns; the counter rises by the number of CTAs;
    the next ordinary call on the same GPU is correct."""
    import torch
    from paper_2609_32237_b200 import binding as B
    n, cols = 4096, 24                       # six tiles, six CTAs
    m = inputs.uniform_complex64((n, cols), 37)
    before = B.tma_timeouts()
    out = run_fft(to_device_c64(m), n, cols, cols, 1, FWD, C64, options={"stream": kind, "starve_wait": 1, "wait_polls": 1024})
    torch.cuda.synchronize()
    assert B.tma_timeouts() - before == 6
    assert bool((out == 0).all())            # nothing was transformed, nothing written
    want = oracle.fft_cols(m.astype(np.complex128), FWD)
    got = run_fft(to_device_c64(m), n, cols, cols, 1, FWD, C64, options={"stream": kind}).cpu().numpy()
    assert np.max(np.linalg.norm(got - want, axis=0) / np.linalg.norm(want, axis=0)) <= TOL32
    assert B.tma_timeouts() - before == 6    # the ordinary call raised nothing


def test_execute_host_pipelined_and_simple_paths():
    """fft_execute_host on pinned host buffers: the chunked, overlapped path (large row
    batch) and the plain path (small batch) both match the device-resident call."""
    import torch
    from paper_2609_32237_b200 import binding as B
    for n, batch in ((1024, 8192), (4096, 6), (32768, 160)):     # the last: the cluster kernel, chunk by chunk
        x = inputs.gaussian_complex64((batch, n), 97)
        h_in = torch.from_numpy(x).pin_memory()
        h_out = torch.zeros_like(h_in).pin_memory()
        d_in = torch.zeros(batch, n, dtype=torch.complex64, device="cuda")
        d_out = torch.zeros_like(d_in)
        plan = B.fft_plan_create(n, batch, 1, n, FWD, C64)
        st = torch.cuda.current_stream().cuda_stream
        for _ in range(2):                      # twice: the second call must wait for the first
            B.fft_execute_host(plan, h_in.data_ptr(), h_out.data_ptr(), d_in.data_ptr(), d_out.data_ptr(), st)
        torch.cuda.synchronize()
        ref = run_fft(to_device_c64(x), n, batch, 1, n, FWD, C64).cpu().numpy()
        B.fft_plan_destroy(plan)
        assert np.array_equal(h_out.numpy().view(np.uint64), ref.view(np.uint64))
        idx = inputs.sample_indices(batch, 8, 3)
        want = oracle.fft_rows(x[idx].astype(np.complex128))
        assert max(worst_rel_l2(h_out.numpy()[idx], want)) <= TOL32


def test_small_batches_pick_the_split_transform_variant():
    """Batches too small to fill the SMs default to a transform split over a cluster of
    CTAs (N = 16384: 4 CTAs up to batch 32, 2 up to 64; N = 8192: 4 CTAs up to batch 32): parity at the
    switch-over sizes."""
    for n, batch in ((16384, 32), (16384, 33), (16384, 64), (16384, 65), (8192, 32), (8192, 33), (16384, 2)):
        _check_rows(n, batch, seed=98, gaussian=True)
        _check_rows(n, batch, seed=99, direction=INV)


def test_seeded_random_plans_against_the_oracle():
    """Forty seeded random plans over sizes, layouts, directions, storage types, ragged
    batches and padded strides; each compared element by element with the oracle."""
    rng = np.random.Generator(np.random.Philox(2024))
    for trial in range(40):
        layout = "rows" if rng.random() < 0.6 else "cols"
        dtype = int(rng.integers(0, 2))
        direction = FWD if rng.random() < 0.5 else INV
        tol = TOL32 if dtype == C64 else TOL16
        if layout == "rows":
            n = int(2 ** rng.integers(8, 15))
            batch = int(rng.integers(1, 10))
            pad = int(rng.integers(0, 3)) * (2 if dtype == C64 else 4)
            dist = n + pad
            x = inputs.gaussian_complex64((batch, dist), 1000 + trial)
            if dtype == C64:
                want = oracle.fft_rows(x[:, :n].astype(np.complex128), direction)
                got = run_fft(to_device_c64(x), n, batch, 1, dist, direction, C64).cpu().numpy()[:, :n]
            else:
                h = inputs.to_half_storage(x)
                want = oracle.fft_rows(inputs.from_half_storage(h)[:, :n], direction)
                got = half_to_c128(run_fft(to_device_half(h), n, batch, 1, dist, direction, C32H))[:, :n]
            worst, pooled = worst_rel_l2(got, want)
        else:
            n = int(2 ** rng.integers(8, 14))
            w = 2 if n == 8192 else 4
            cols = w * int(rng.integers(1, 5))
            ld = cols + int(rng.integers(0, 3)) * 4
            m = inputs.uniform_complex64((n, ld), 2000 + trial)
            if dtype == C64:
                want = oracle.fft_cols(m[:, :cols].astype(np.complex128), direction)
                got = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64).cpu().numpy()[:, :cols]
            else:
                h = inputs.to_half_storage(m)
                want = oracle.fft_cols(inputs.from_half_storage(h)[:, :cols], direction)
                got = half_to_c128(run_fft(to_device_half(h), n, cols, ld, 1, direction, C32H))[:, :cols]
            worst = pooled = rel_l2(got, want)
        assert worst <= tol and pooled <= tol, (trial, layout, n, dtype, direction, worst)


@pytest.mark.parametrize("n", [8, 16, 32, 64, 128])
def test_small_transforms(n):
    """N = 8 ... 128: several transforms per CTA (one thread per transform at N = 8 and 16), ragged
    batches, both directions, padding, fp16 storage; each against the direct DFT."""
    for batch in (1, 5, 130, 1000):
        _check_rows(n, batch, seed=300 + n + batch, gaussian=(batch == 130))
        _check_rows(n, batch, seed=301 + n + batch, direction=INV)
    _check_rows(n, 37, seed=302, dist=n + 6)
    x = inputs.gaussian_complex64((77, n), 303)
    h = inputs.to_half_storage(x)
    want = oracle.fft_rows(inputs.from_half_storage(h), FWD)
    got = half_to_c128(run_fft(to_device_half(h), n, 77, 1, n, FWD, C32H))
    assert max(worst_rel_l2(got, want)) <= TOL16


@pytest.mark.parametrize("n", [8, 16, 32])
def test_tiny_transforms_both_kernels(n):
    """N <= 32 on a contiguous batch runs the chunk-staging kernel by default (one thread per transform,
    128 transforms per CTA through shared memory) and the plain kernel with staged = 0: both against the
    direct DFT, batches that end inside a CTA's chunk, in place, both directions and storage types."""
    for batch in (1, 127, 128, 129, 1000, 4099):
        for direction in (FWD, INV):
            x = inputs.gaussian_complex64((batch, n), 310 + n + batch)
            want = oracle.fft_rows(x.astype(np.complex128), direction)
            for options in (None, {"staged": 0}):
                got = run_fft(to_device_c64(x), n, batch, 1, n, direction, C64, options=options).cpu().numpy()
                assert max(worst_rel_l2(got, want)) <= TOL32, (n, batch, direction, options)
            got = run_fft(to_device_c64(x), n, batch, 1, n, direction, C64, inplace=True).cpu().numpy()
            assert max(worst_rel_l2(got, want)) <= TOL32
            h = inputs.to_half_storage(x)
            want16 = oracle.fft_rows(inputs.from_half_storage(h), direction)
            for options in (None, {"staged": 0}):
                got = half_to_c128(run_fft(to_device_half(h), n, batch, 1, n, direction, C32H, options=options))
                assert max(worst_rel_l2(got, want16)) <= TOL16, (n, batch, direction, options)


@pytest.mark.parametrize("n,batch", [(16384, 5), (16384, 300), (16384, 449)])
@pytest.mark.parametrize("dtype", [C64, C32H])
def test_staged_persistent_rows(n, batch, dtype):
    """The persistent row kernel whose next tile arrives through the copy engine while the
    current one is transformed: fewer tiles than CTAs, several tiles per CTA with a ragged
    last round, both directions and storage types; no bounded wait ran out."""
    from paper_2609_32237_b200 import binding as B
    x = inputs.gaussian_complex64((batch, n), 300 + batch)
    rows = inputs.sample_indices(batch, 6, seed=batch)
    for direction in (FWD, INV):
        if dtype == C64:
            got = run_fft(to_device_c64(x), n, batch, 1, n, direction, C64, options={"staged": 1}).cpu().numpy()
            xin, tol = x.astype(np.complex128), TOL32
        else:
            h = inputs.to_half_storage(x)
            got = half_to_c128(run_fft(to_device_half(h), n, batch, 1, n, direction, C32H, options={"staged": 1}))
            xin, tol = inputs.from_half_storage(h), TOL16
        want = oracle.fft_rows(xin[rows], direction)
        assert max(worst_rel_l2(got[rows], want)) <= tol
        assert np.isfinite(np.abs(got)).all()
    assert B.tma_timeouts() == _timeouts_at_start(B)


def test_staged_rows_default_choice_and_other_sizes():
    """fp16 storage at n = 16384 takes the staged kernel by default once every multiprocessor
    has two transforms: same network, so the result equals the plain kernel's to the last digit.
    Sizes without a staged variant refuse the option and keep working."""
    import torch
    from paper_2609_32237_b200 import binding as B
    n, batch = 16384, 300
    h = inputs.to_half_storage(inputs.gaussian_complex64((batch, n), 77))
    a = run_fft(to_device_half(h), n, batch, 1, n, FWD, C32H).cpu().numpy()
    b = run_fft(to_device_half(h), n, batch, 1, n, FWD, C32H, options={"staged": 0}).cpu().numpy()
    # same network, separately compiled: equal up to the last fp16 digit of a few elements
    assert np.mean(a.view(np.uint16) != b.view(np.uint16)) < 1e-3
    assert rel_l2(half_to_c128(torch.from_numpy(a)), half_to_c128(torch.from_numpy(b))) <= 1e-4
    plan = B.fft_plan_create(4096, 8, 1, 4096, FWD, C64)
    try:
        with pytest.raises(B.B200FftError) as e:
            B.fft_plan_set_option(plan, "staged", 1)
        assert e.value.status == 2
        x4 = inputs.gaussian_complex64((8, 4096), 5)                 # the plan still works afterwards
        d = to_device_c64(x4)
        o = torch.zeros_like(d)
        B.fft_execute(plan, d.data_ptr(), o.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert max(worst_rel_l2(o.cpu().numpy(), oracle.fft_rows(x4.astype(np.complex128), FWD))) <= TOL32
    finally:
        B.fft_plan_destroy(plan)
    assert B.tma_timeouts() == _timeouts_at_start(B)


@pytest.mark.parametrize("n,cols,ld", [(1024, 24, 24), (4096, 68, 72), (256, 36, 40)])
def test_columns_via_transpose(n, cols, ld):
    """A columns plan run as transpose + row transforms + transpose back (the paper's four-pass
    form): same results as the oracle and as the direct column kernel, padding untouched,
    both storage types and directions; the workspace is required."""
    import torch
    from paper_2609_32237_b200 import binding as B
    m = inputs.uniform_complex64((n, ld), 61)
    for direction in (FWD, INV):
        want = oracle.fft_cols(m[:, :cols].astype(np.complex128), direction)
        got = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64, options={"via_transpose": 1}).cpu().numpy()
        direct = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64).cpu().numpy()
        per_col = np.linalg.norm(got[:, :cols] - want, axis=0) / np.linalg.norm(want, axis=0)
        assert per_col.max() <= TOL32
        assert rel_l2(got[:, :cols], direct[:, :cols]) <= 1e-6
        assert np.all(got[:, cols:] == 0)
    h = inputs.to_half_storage(m)
    want = oracle.fft_cols(inputs.from_half_storage(h)[:, :cols], FWD)
    got = half_to_c128(run_fft(to_device_half(h), n, cols, ld, 1, FWD, C32H, options={"via_transpose": 1}))
    assert rel_l2(got[:, :cols], want) <= TOL16
    plan = B.fft_plan_create(n, cols, ld, 1, FWD, C64)
    try:
        B.fft_plan_set_option(plan, "via_transpose", 1)
        assert B.fft_plan_workspace_bytes(plan) == n * cols * 8
        d = to_device_c64(m)
        with pytest.raises(B.B200FftError) as e:
            B.fft_execute(plan, d.data_ptr(), d.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert e.value.status == 6
    finally:
        B.fft_plan_destroy(plan)
    rows_plan = B.fft_plan_create(n, 4, 1, n, FWD, C64)
    try:
        with pytest.raises(B.B200FftError) as e:
            B.fft_plan_set_option(rows_plan, "via_transpose", 1)
        assert e.value.status == 2
    finally:
        B.fft_plan_destroy(rows_plan)


@pytest.mark.parametrize("n,cols,ld", [(256, 32, 40), (512, 16, 16), (1024, 24, 24), (1024, 40, 48), (64, 48, 52),
                                       (128, 16, 16), (64, 20, 20), (128, 4, 4)])
def test_columns_wide_tiles_by_default(n, cols, ld):
    """Short column transforms whose batch is a multiple of the wide tile (16 columns, 8 at
    n = 1024) take it by default: checked against the oracle and the narrow-tile kernel
    (option cluster = 1), both directions and storage types, padding untouched."""
    m = inputs.uniform_complex64((n, ld), 62)
    for direction in (FWD, INV):
        want = oracle.fft_cols(m[:, :cols].astype(np.complex128), direction)
        got = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64).cpu().numpy()
        narrow = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64, options={"cluster": 1}).cpu().numpy()
        per_col = np.linalg.norm(got[:, :cols] - want, axis=0) / np.linalg.norm(want, axis=0)
        assert per_col.max() <= TOL32
        assert rel_l2(got[:, :cols], narrow[:, :cols]) <= 1e-6
        assert np.all(got[:, cols:] == 0)
    h = inputs.to_half_storage(m)
    want = oracle.fft_cols(inputs.from_half_storage(h)[:, :cols], FWD)
    got = half_to_c128(run_fft(to_device_half(h), n, cols, ld, 1, FWD, C32H))
    assert rel_l2(got[:, :cols], want) <= TOL16


def test_n32768_runs_in_one_pass_on_a_cluster_of_two():
    """n = 32768 does not fit one CTA; by default two CTAs of a cluster share the transform
    through distributed shared memory, in one pass and without a workspace. Checked against
    the oracle and the two-pass split, ragged batch, both directions and storage types."""
    from paper_2609_32237_b200 import binding as B
    n, batch = 32768, 7
    plan = B.fft_plan_create(n, batch, 1, n, FWD, C64)
    try:
        assert B.fft_plan_workspace_bytes(plan) == 0
        B.fft_plan_set_option(plan, "four_step", 1)
        assert B.fft_plan_workspace_bytes(plan) == n * batch * 8
        B.fft_plan_set_option(plan, "four_step", 0)
        assert B.fft_plan_workspace_bytes(plan) == 0
    finally:
        B.fft_plan_destroy(plan)
    x = inputs.gaussian_complex64((batch, n + 6), 321)[:, :]
    for direction in (FWD, INV):
        want = oracle.fft_rows(x[:, :n].astype(np.complex128), direction)
        got = run_fft(to_device_c64(x), n, batch, 1, n + 6, direction, C64).cpu().numpy()       # padded rows
        two = run_fft(to_device_c64(x), n, batch, 1, n + 6, direction, C64, options={"four_step": 1}).cpu().numpy()
        assert max(worst_rel_l2(got[:, :n], want)) <= TOL32
        assert rel_l2(got[:, :n], two[:, :n]) <= 1e-6
        assert np.all(got[:, n:] == 0)
    h = inputs.to_half_storage(np.ascontiguousarray(x[:, :n]))
    want = oracle.fft_rows(inputs.from_half_storage(h), FWD)
    got = half_to_c128(run_fft(to_device_half(h), n, batch, 1, n, FWD, C32H))
    assert max(worst_rel_l2(got, want)) <= TOL16
    # in place: both CTAs of a cluster have read their inputs before either stores (cluster barrier)
    xc = np.ascontiguousarray(x[:, :n])
    inplace = run_fft(to_device_c64(xc), n, batch, 1, n, FWD, C64, inplace=True).cpu().numpy()
    outplace = run_fft(to_device_c64(xc), n, batch, 1, n, FWD, C64).cpu().numpy()
    assert np.array_equal(inplace.view(np.uint64), outplace.view(np.uint64))


def test_execute_host_with_fp16_storage_and_the_staged_kernel():
    """The chunked host path on fp16 storage at n = 16384, where the persistent staged kernel is the
    default and every chunk is one launch of it with fewer tiles than CTAs."""
    import torch
    from paper_2609_32237_b200 import binding as B
    n, batch = 16384, 640
    h = inputs.to_half_storage(inputs.gaussian_complex64((batch, n), 98))
    h_in = torch.from_numpy(h).pin_memory()
    h_out = torch.zeros_like(h_in).pin_memory()
    d_in = torch.zeros(batch, n, 2, dtype=torch.float16, device="cuda")
    d_out = torch.zeros_like(d_in)
    plan = B.fft_plan_create(n, batch, 1, n, FWD, C32H)
    try:
        B.fft_execute_host(plan, h_in.data_ptr(), h_out.data_ptr(), d_in.data_ptr(), d_out.data_ptr(),
                           torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
    finally:
        B.fft_plan_destroy(plan)
    idx = inputs.sample_indices(batch, 6, 4)
    want = oracle.fft_rows(inputs.from_half_storage(h[idx]), FWD)
    assert max(worst_rel_l2(half_to_c128(h_out[torch.from_numpy(idx)]), want)) <= TOL16
    assert B.tma_timeouts() == _timeouts_at_start(B)


@pytest.mark.parametrize("n,cols,ld", [(4096, 24, 26), (4096, 8, 8), (8192, 12, 12), (8192, 4, 6), (2048, 32, 36)])
def test_columns_wider_tiles_on_a_cluster_by_default(n, cols, ld):
    """n = 4096 with a batch that is a multiple of 8, n = 8192 with a multiple of 4: the default is
    a tile twice as wide shared by a cluster of two CTAs (64- resp. 32-byte row segments). Checked
    against the oracle and the single-CTA tile (option cluster = 1), both directions and storage
    types, padding untouched."""
    m = inputs.uniform_complex64((n, ld), 63)
    for direction in (FWD, INV):
        want = oracle.fft_cols(m[:, :cols].astype(np.complex128), direction)
        got = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64).cpu().numpy()
        narrow = run_fft(to_device_c64(m), n, cols, ld, 1, direction, C64, options={"cluster": 1}).cpu().numpy()
        per_col = np.linalg.norm(got[:, :cols] - want, axis=0) / np.linalg.norm(want, axis=0)
        assert per_col.max() <= TOL32
        assert rel_l2(got[:, :cols], narrow[:, :cols]) <= 1e-6
        assert np.all(got[:, cols:] == 0)
    if ld % 4 == 0:                                     # fp16 storage wants rows that are multiples of 16 bytes
        h = inputs.to_half_storage(m)
        want = oracle.fft_cols(inputs.from_half_storage(h)[:, :cols], FWD)
        got = half_to_c128(run_fft(to_device_half(h), n, cols, ld, 1, FWD, C32H))
        assert rel_l2(got[:, :cols], want) <= TOL16
