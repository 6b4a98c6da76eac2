"""Pins for the float64 range-Doppler oracle: closed forms for single steps,
the simulator's independent geometry, the values the paper prints for its
worked scene, and the ablations the paper describes."""
import math

import numpy as np
import pytest

import oracle
from oracle import quality
from paper_2609_32237_b200 import inputs

from conftest import read_golden


def _rel(a, b):
    return np.linalg.norm(np.asarray(a) - np.asarray(b)) / np.linalg.norm(np.asarray(b))


# --- range compression: closed form ------------------------------------------------
def test_range_compression_of_an_on_grid_echo_closed_form():
    """One noise-free echo whose delay is on the sample grid: the compressed
    pulse is the sampled chirp's autocorrelation, a geometric sum:
    |y[n_t + d]| = |sin(pi kappa d (P - |d|)) / sin(pi kappa d)|, kappa = K / fs^2,
    P = 1200 samples, and exactly P at d = 0."""
    sc = inputs.x_band_scene(n_azimuth=4, n_range=4096, n_targets=0)
    P = sc.pulse_samples
    assert P == 1200
    n_t = 1777
    kappa = sc.chirp_rate / sc.fs_hz ** 2
    raw = np.zeros((4, 4096), dtype=np.complex128)
    i = np.arange(-P // 2, P // 2)
    raw[1, n_t + i] = np.exp(1j * np.pi * kappa * i.astype(np.float64) ** 2)
    p = oracle.sar_params(sc)
    y = oracle.sar_range_compress(p, raw)
    assert np.abs(y[0]).max() < 1e-9 and np.abs(y[2]).max() < 1e-9
    assert abs(y[1, n_t] - P) < 1e-9                     # real, positive, exactly the pulse length
    d = np.arange(-1300, 1301)
    with np.errstate(invalid="ignore", divide="ignore"):
        want = np.abs(np.sin(np.pi * kappa * d * (P - np.abs(d))) / np.sin(np.pi * kappa * d))
    want[d == 0] = P
    want[np.abs(d) >= P] = 0.0
    np.testing.assert_allclose(np.abs(y[1, n_t + d]), want, atol=1e-8)


def test_matched_filter_has_unit_dc_free_structure():
    sc = inputs.x_band_scene(n_azimuth=4, n_range=4096, n_targets=0)
    H = oracle.sar_matched_filter(oracle.sar_params(sc))
    # Parseval on the replica: sum |H|^2 = N * P
    assert abs((np.abs(H) ** 2).sum() - 4096 * 1200) < 1e-6
    # the in-band plateau of a large time-bandwidth chirp is about sqrt(fs^2 / K)
    assert abs(np.median(np.abs(H[:1000])) - math.sqrt(sc.fs_hz ** 2 / sc.chirp_rate)) < 2.0


# --- interpolator ---------------------------------------------------------------------
def test_interpolator_weights():
    w0 = oracle.sar_interp_weights(0.0)
    np.testing.assert_allclose(w0, [0, 0, 0, 1, 0, 0, 0, 0], atol=1e-15)   # tap j=0 is index 3
    for mu in (0.1, 0.37, 0.5, 0.93):
        w = oracle.sar_interp_weights(mu)
        assert abs(w.sum() - 1.0) < 1e-15
        # the two taps that bracket the position carry the weight; mu < .5 favours j=0
        assert (w[3] > w[4]) == (mu < 0.5)
        # signs alternate away from the bracketing pair
        assert w[2] < 0 < w[1] and w[5] < 0 < w[6]
    a, b = oracle.sar_interp_weights(0.3), oracle.sar_interp_weights(0.7)
    # w_j(mu) = w_{1-j}(1-mu): taps -3..4 map onto 4..-3
    np.testing.assert_allclose(a, b[::-1], atol=1e-15)
    # continuity across an integer: mu -> 1 from below equals mu = 0 one sample on
    c = oracle.sar_interp_weights(1.0 - 1e-9)
    np.testing.assert_allclose(c, [0, 0, 0, 0, 1, 0, 0, 0], atol=1e-8)


def test_rcmc_shifts_a_smooth_row_by_the_migration():
    """A slowly varying band-limited row, resampled by the oracle, equals the row
    evaluated at n + dn(k, n) to the accuracy of an 8-tap truncated sinc."""
    sc = inputs.x_band_scene(n_azimuth=8, n_range=4096, n_targets=0)
    sc.prf_hz = 1000.0
    p = oracle.sar_params(sc)
    n = np.arange(4096, dtype=np.float64)
    f0 = 0.031                                  # cycles per sample, well inside the band
    S = np.tile(np.exp(2j * np.pi * f0 * n), (8, 1))
    out = oracle.sar_rcmc(p, S)
    for k in (0, 3, 4, 7):
        dn = np.array([oracle.sar_migration_bins(p, k, int(c)) for c in range(4096)])
        want = np.exp(2j * np.pi * f0 * (n + dn))
        mid = slice(16, 4096 - 16)
        # an unwindowed 8-tap sinc has a few per cent of pass-band ripple in gain,
        # but it places the samples at the right position: the phase agrees closely
        assert np.abs(out[k, mid] - want[mid]).max() < 6e-2
        assert np.abs(np.angle(out[k, mid] * np.conj(want[mid]))).max() < 5e-3
    # zero Doppler: no migration, rows pass through untouched
    assert oracle.sar_migration_bins(p, 0, 100) == 0.0
    np.testing.assert_allclose(out[0], S[0], atol=1e-15)


# --- migration and phase: the simulator's geometry pins the processor's formulas ----
@pytest.fixture(scope="module")
def single_target_xband():
    sc = inputs.x_band_scene(n_azimuth=4096, n_range=2048, n_targets=0)
    sc.targets = [(2048, 1100)]
    sc.noise_variance = 0.0
    raw = inputs.simulate_raw(sc, dtype=np.complex128)
    p = oracle.sar_params(sc)
    img, rc = oracle.sar_rda(p, raw, want_range_compressed=True)
    return sc, p, raw, rc, img


def _ridge(S, k, n_t):
    """Energy centroid of the range-Doppler spectrum of one target along range, Doppler bin k."""
    cols = np.arange(n_t - 12, n_t + 20)
    prof = np.abs(S[k, cols]) ** 2
    return (prof * cols).sum() / prof.sum()


def test_migration_formula_follows_the_simulated_trajectory(single_target_xband):
    """The simulator moves the echo along sqrt(R^2 + v^2 eta^2); in the
    range-Doppler domain its ridge must sit at n_t + dn(k, n_t). The Doppler
    bins reach to 244 Hz of the 267 Hz half band, where the ridge has moved by
    a bin and a half, so a missing or mis-scaled migration term fails."""
    sc, p, raw, rc, img = single_target_xband
    a_t, n_t = sc.targets[0]
    assert abs(abs(rc[a_t, n_t]) - 1200) < 1e-6          # on-grid at closest approach
    S = oracle.sar_azimuth_fft(p, rc)
    for k in (0, 40, 120, 200, 600, 1000, 4096 - 1000, 4096 - 600, 4096 - 200, 4096 - 60):
        assert abs(_ridge(S, k, n_t) - (n_t + oracle.sar_migration_bins(p, k, n_t))) < 0.05
    # the ridge itself, with no formula involved: it has left the target's bin by more than a bin
    assert _ridge(S, 1000, n_t) - _ridge(S, 0, n_t) > 1.0
    assert _ridge(S, 4096 - 1000, n_t) - _ridge(S, 0, n_t) > 1.0
    assert 0.4 < _ridge(S, 600, n_t) - _ridge(S, 0, n_t) < 0.7
    # a formula that returned no migration would miss the ridge by far more than the tolerance
    assert abs(_ridge(S, 1000, n_t) - n_t) > 1.0


def test_interpolator_hand_values_at_half_a_sample():
    """mu = 1/2: sinc(1/2 - j) = (-1)^j / (pi (1/2 - j)), so the eight taps j = -3 .. 4 are
    proportional to -1/7, 1/5, -1/3, 1, 1, -1/3, 1/5, -1/7 and sum to one."""
    pattern = np.array([-1 / 7, 1 / 5, -1 / 3, 1.0, 1.0, -1 / 3, 1 / 5, -1 / 7])
    np.testing.assert_allclose(oracle.sar_interp_weights(0.5), pattern / pattern.sum(), atol=1e-15)
    # any fraction, against the library's sinc
    for mu in (0.0, 0.125, 0.3, 0.77):
        w = np.sinc(mu - np.arange(-3, 5))
        np.testing.assert_allclose(oracle.sar_interp_weights(mu), w / w.sum(), atol=1e-15)


@pytest.mark.parametrize("band", ["x", "l"])
def test_rcmc_of_an_impulse_row_lays_out_the_taps_in_order(band):
    """A row that is delta[n - n1] comes out as S'[k, n] = w_j(mu(k, n)) at n = n1 - i0 - j: the
    eight weights in REVERSED tap order around n1 - i0 (tap j = 4 first), nothing elsewhere. This
    fixes the tap orientation and the index convention n + i0 + j exactly; on the L-band scene the
    integer shift is over a hundred bins."""
    if band == "x":
        sc = inputs.x_band_scene(n_azimuth=64, n_range=2048, n_targets=0)
        ks, n1 = (0, 9, 17, 31, 33, 50), 1000
    else:
        sc = inputs.l_band_scene(n_azimuth=64, n_range=2048, targets=[])
        ks, n1 = (0, 5, 22, 31, 32, 40), 1300
    p = oracle.sar_params(sc)
    S = np.zeros((64, 2048), dtype=np.complex128)
    S[:, n1] = 1.0 + 0.5j
    out = oracle.sar_rcmc(p, S)
    lam, dr = sc.wavelength_m, sc.range_bin_m
    biggest = 0
    for k in ks:
        f = (k if k < 32 else k - 64) * sc.prf_hz / 64
        d = math.sqrt(1.0 - (lam * f / (2.0 * sc.velocity_mps)) ** 2)
        want = np.zeros(2048, dtype=np.complex128)
        for n in range(2048):
            dn = (sc.r_center_m + (n - 1024) * dr) * (1.0 / d - 1.0) / dr
            i0 = math.floor(dn)
            j = n1 - n - i0
            if -3 <= j <= 4:
                w = np.sinc((dn - i0) - np.arange(-3, 5))
                want[n] = (1.0 + 0.5j) * w[j + 3] / w.sum()
                biggest = max(biggest, i0)
        assert np.count_nonzero(want) == 8
        np.testing.assert_allclose(out[k], want, atol=1e-9)
        if k == 0:
            assert out[k, n1] == 1.0 + 0.5j                      # no migration at zero Doppler
        else:
            # mirrored taps would swap the two unequal neighbours of the main tap
            nz = np.nonzero(want)[0]
            assert abs(abs(want[nz[3]]) - abs(want[nz[4]])) > 1e-3 or abs(abs(want[nz[2]]) - abs(want[nz[5]])) > 1e-4
    assert biggest >= (100 if band == "l" else 5)


def test_target_focuses_at_its_cell_with_textbook_quality(single_target_xband):
    sc, p, raw, rc, img = single_target_xband
    cell = tuple(sc.targets[0])
    assert quality.peak_cell(img, cell) == cell
    wr, pr, off_r = quality.irw_pslr(quality.cut_through(img, cell, 1))
    wa, pa, off_a = quality.irw_pslr(quality.cut_through(img, cell, 0))
    assert abs(off_r) < 0.04 and abs(off_a) < 0.04
    assert abs(wr - 0.886 * sc.fs_hz / sc.bandwidth_hz) < 0.02            # 1.063 bins
    dopp_bw = 2 * sc.velocity_mps / sc.antenna_m
    assert abs(wa - 0.886 * sc.prf_hz / dopp_bw) < 0.05                    # 1.66 bins
    assert abs(pr + 13.26) < 0.5 and abs(pa + 13.26) < 1.0
    # the filter removes the Doppler phase history and leaves the two-way carrier
    # phase at closest approach plus the stationary-phase constant of the
    # azimuth down-chirp: arg(peak) = -4 pi R_t / lambda - pi/4
    r_t = sc.r_center_m + (cell[1] - sc.n_range // 2) * sc.range_bin_m
    want = (-4 * math.pi * r_t / sc.wavelength_m - math.pi / 4) % (2 * math.pi)
    got = np.angle(img[cell]) % (2 * math.pi)
    assert abs((got - want + math.pi) % (2 * math.pi) - math.pi) < 0.05


def test_ablations(single_target_xband):
    sc, p, raw, rc, img = single_target_xband
    cell = tuple(sc.targets[0])
    # migration correction off: the peak drops and the range response broadens
    p_off = oracle.sar_params(sc, rcmc_enabled=False)
    img_off = oracle.sar_rda(p_off, raw)
    assert np.abs(img_off).max() < 0.75 * np.abs(img).max()
    pk = np.unravel_index(np.argmax(np.abs(img_off)), img_off.shape)
    w_off = quality.irw_pslr(quality.cut_through(img_off, pk, 1))[0]
    w_on = quality.irw_pslr(quality.cut_through(img, cell, 1))[0]
    assert w_off > w_on + 0.1
    # textbook filter with D instead of (D - 1): same image magnitude (first fix)
    p_d = oracle.sar_params(sc, baseband_filter=False)
    img_d = oracle.sar_rda(p_d, raw)
    assert _rel(np.abs(img_d), np.abs(img)) < 1e-8
    assert _rel(img_d, img) > 0.1                                            # but not the same phase
    # the azimuth filter is a pure phase: it keeps every sample's magnitude
    S1 = oracle.sar_rcmc(p, oracle.sar_azimuth_fft(p, rc))
    S2 = oracle.sar_azimuth_filter(p, S1)
    np.testing.assert_allclose(np.abs(S2), np.abs(S1), rtol=1e-12, atol=1e-12)


# --- the paper's worked scene ---------------------------------------------------------
def test_paper_scene_numbers():
    g = read_golden("paper_sar_scene.txt")
    sc = inputs.l_band_scene(n_azimuth=4096, n_range=2048, targets=[(2048, 1024), (1500, 800)])
    assert abs(sc.wavelength_m - 0.24) < 1e-12
    p = oracle.sar_params(sc)
    # aperture and migration across it, from the simulator's geometry alone
    aperture = sc.wavelength_m * sc.r_center_m / sc.antenna_m
    assert abs(aperture - g["aperture_m"]) < 1.0
    rcm = (math.hypot(sc.r_center_m, aperture / 2) - sc.r_center_m) / sc.range_bin_m
    assert abs(rcm - g["range_migration_bins"]) < 0.05
    # phase slope the textbook filter would add per range bin, and the baseband
    # filter's phase at the band edge
    per_bin = abs(oracle.sar_filter_phase(oracle.sar_params(sc, baseband_filter=False), 0, 1025)
                  - oracle.sar_filter_phase(oracle.sar_params(sc, baseband_filter=False), 0, 1024))
    assert abs(per_bin - g["phase_per_range_bin_rad"]) < 0.5
    edge = abs(oracle.sar_filter_phase(p, 2048, 1024))
    assert 0.8 * g["phase_at_half_prf_rad"] < edge < 1.5 * g["phase_at_half_prf_rad"]
    # the focused image
    raw = inputs.simulate_raw(sc, dtype=np.complex128)
    img = oracle.sar_rda(p, raw)
    for cell in sc.targets:
        cell = tuple(cell)
        assert quality.peak_cell(img, cell) == cell
        wr, pr, _ = quality.irw_pslr(quality.cut_through(img, cell, 1))
        wa, pa, _ = quality.irw_pslr(quality.cut_through(img, cell, 0, half=128))
        assert abs(wr - g["irw_range_bins"]) < 0.02
        assert abs(wa - g["irw_azimuth_bins"]) < 0.1
        assert abs(wa - g["irw_azimuth_theory"]) < 0.15
        assert abs(pr - g["pslr_range_db"]) < 0.3
        assert abs(pa - g["pslr_theory_db"]) < 1.0


def test_multi_target_scene_with_noise_focuses_every_target():
    sc = inputs.x_band_scene(n_azimuth=4096, n_range=2048, n_targets=6, seed=4)
    raw = inputs.simulate_raw(sc, seed=4)
    assert raw.dtype == np.complex64
    img = oracle.sar_rda(oracle.sar_params(sc), raw)
    for cell in sc.targets:
        assert quality.peak_cell(img, tuple(cell)) == tuple(cell)
    # noise at 20 dB below a unit echo: raw noise variance 0.01 (0.005 per component)
    quiet = raw[:64, :64]
    if np.abs(quiet).max() < 1.0:                       # no echo in that corner
        assert abs(quiet.real.var() - 0.005) < 5e-4
