"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA path.

This module holds NO arithmetic of the method (no FFT, no range-Doppler step).
It only manufactures inputs: random batches with the value distributions the
paper's workloads use (Section "Platform and Methodology": random inputs,
uniform on [-1, 1]) and a simulated stripmap point-target raw-data matrix
(Section "End to End: Range-Doppler SAR": point targets plus complex Gaussian
noise, rectangular beam, flat earth, zero squint).

Everything is generated on the host with numpy's counter-based Philox
generator, so a (seed, shape) pair names one bit pattern on every machine.
"""
from __future__ import annotations

from dataclasses import dataclass, field, asdict
import numpy as np

C_LIGHT = 299_792_458.0  # m/s


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed)))


def uniform_complex64(shape, seed: int) -> np.ndarray:
    """Real and imaginary parts i.i.d. uniform on [-1, 1), float64 draw rounded
    once to fp32 (a draw that rounds up to 1.0 is pulled back to the largest
    fp32 below 1)."""
    g = _rng(seed)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.complex64)
    v = out.view(np.float32)
    chunk = 1 << 24
    for s in range(0, 2 * n, chunk):
        e = min(2 * n, s + chunk)
        d = g.random(e - s) * 2.0 - 1.0
        f = d.astype(np.float32)
        np.minimum(f, np.nextafter(np.float32(1.0), np.float32(0.0)), out=f)
        v[s:e] = f
    return out.reshape(shape)


def gaussian_complex64(shape, seed: int, sigma: float = 1.0) -> np.ndarray:
    """Real and imaginary parts i.i.d. N(0, sigma^2) each (so the complex
    variance is 2 sigma^2), drawn directly in fp32."""
    g = _rng(seed)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.complex64)
    v = out.view(np.float32)
    chunk = 1 << 24
    for s in range(0, 2 * n, chunk):
        e = min(2 * n, s + chunk)
        v[s:e] = g.standard_normal(e - s, dtype=np.float32)
    if sigma != 1.0:
        v *= np.float32(sigma)
    return out.reshape(shape)


def to_half_storage(x: np.ndarray) -> np.ndarray:
    """complex64 -> interleaved fp16 pairs, shape (..., 2), round to nearest even."""
    v = np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,))
    return v.astype(np.float16)


def from_half_storage(h: np.ndarray) -> np.ndarray:
    """Interleaved fp16 pairs (..., 2) -> complex128, exact."""
    d = h.astype(np.float64)
    return d[..., 0] + 1j * d[..., 1]


def sample_indices(batch: int, count: int, seed: int) -> np.ndarray:
    """First 4, last 4 and seeded random transform indices (sorted, unique)."""
    fixed = list(range(min(4, batch))) + list(range(max(0, batch - 4), batch))
    g = _rng(seed)
    extra = g.integers(0, batch, size=max(0, count - len(fixed))).tolist()
    return np.array(sorted(set(fixed + extra)), dtype=np.int64)


# ----------------------------------------------------------------------------
# SAR scenes
# ----------------------------------------------------------------------------
@dataclass
class SarScene:
    """Radar and geometry parameters of a stripmap scene; plain numbers only."""
    n_azimuth: int = 4096
    n_range: int = 4096
    carrier_hz: float = 9.6e9
    bandwidth_hz: float = 100e6
    fs_hz: float = 120e6
    pulse_s: float = 10e-6
    prf_hz: float = 1000.0
    velocity_mps: float = 200.0
    r_center_m: float = 10_000.0
    antenna_m: float = 0.75           # simulator only: sets the beam-limited aperture
    noise_variance: float = 0.01      # total complex variance; 20 dB below a unit echo
    targets: list = field(default_factory=list)  # (azimuth_cell, range_cell) integer pairs

    @property
    def wavelength_m(self) -> float:
        return C_LIGHT / self.carrier_hz

    @property
    def range_bin_m(self) -> float:
        return C_LIGHT / (2.0 * self.fs_hz)

    @property
    def chirp_rate(self) -> float:
        return self.bandwidth_hz / self.pulse_s

    @property
    def pulse_samples(self) -> int:
        return int(round(self.pulse_s * self.fs_hz))

    def as_dict(self):
        return asdict(self)


def x_band_scene(n_azimuth=4096, n_range=4096, n_targets=16, seed=4) -> SarScene:
    """The measured scene: 9.6 GHz carrier, 100 MHz chirp sampled at 120 MHz,
    10 us pulse, PRF 1 kHz, 200 m/s, 10 km scene centre; unit point targets at
    seeded integer cells, kept far enough from the frame edge that the whole
    aperture and the whole pulse stay inside it."""
    sc = SarScene(n_azimuth=n_azimuth, n_range=n_range)
    sc.targets = seeded_target_cells(sc, n_targets, seed) if n_targets > 0 else []
    return sc


def l_band_scene(n_azimuth=4096, n_range=4096, targets=None) -> SarScene:
    """The paper's worked scene (Section "End to End"): wavelength 0.24 m,
    100 MHz bandwidth, 120 MHz sampling, 200 m/s, PRF 500 Hz, 8 m antenna.
    A 20 km scene-centre range reproduces the 600 m aperture and the 1.8-bin
    range migration the paper states."""
    sc = SarScene(n_azimuth=n_azimuth, n_range=n_range,
                  carrier_hz=C_LIGHT / 0.24, prf_hz=500.0, antenna_m=8.0,
                  r_center_m=20_000.0, noise_variance=0.0)
    sc.targets = list(targets) if targets is not None else [(n_azimuth // 2, n_range // 2)]
    return sc


def target_box(sc: SarScene):
    """Cells whose full synthetic aperture and full pulse lie inside the frame."""
    half_pulse = sc.pulse_samples // 2
    r_far = sc.r_center_m + (sc.n_range / 2) * sc.range_bin_m
    half_ap = int(np.ceil(0.5 * sc.wavelength_m * r_far / sc.antenna_m
                          / sc.velocity_mps * sc.prf_hz))
    # migration at the aperture edge moves the echo a few bins further out
    guard = 40
    return (half_ap + guard, sc.n_azimuth - half_ap - guard,
            half_pulse + guard, sc.n_range - half_pulse - guard)


def seeded_target_cells(sc: SarScene, count: int, seed: int, min_sep: int = 64):
    """Integer (azimuth, range) cells by seeded rejection sampling, pairwise
    Chebyshev distance >= min_sep."""
    a0, a1, r0, r1 = target_box(sc)
    if a1 <= a0 or r1 <= r0:
        raise ValueError("frame too small for a full aperture and pulse")
    g = _rng(seed)
    cells = []
    tries = 0
    while len(cells) < count:
        tries += 1
        if tries > 100000:
            raise RuntimeError("could not place targets")
        a = int(g.integers(a0, a1 + 1))
        r = int(g.integers(r0, r1 + 1))
        if all(max(abs(a - pa), abs(r - pr)) >= min_sep for pa, pr in cells):
            cells.append((a, r))
    return cells


def simulate_raw(sc: SarScene, seed: int = 4, dtype=np.complex64) -> np.ndarray:
    """Raw echo matrix raw[m, n] (pulse m, range sample n) of unit point
    targets: for each pulse inside the target's beam-limited aperture, the
    delayed linear-FM pulse times the two-way carrier phase; then additive
    complex Gaussian noise. Accumulated in float64, rounded once to `dtype`."""
    na, nr = sc.n_azimuth, sc.n_range
    lam, dr, K, fs = sc.wavelength_m, sc.range_bin_m, sc.chirp_rate, sc.fs_hz
    half = sc.pulse_samples / 2.0
    raw = np.zeros((na, nr), dtype=np.complex128)
    eta = (np.arange(na) - na // 2) / sc.prf_hz
    ncol = np.arange(nr, dtype=np.float64) - nr // 2
    for (ma, nrg) in sc.targets:
        r_t = sc.r_center_m + (nrg - nr // 2) * dr
        eta_t = (ma - na // 2) / sc.prf_hz
        l_s = lam * r_t / sc.antenna_m
        x = sc.velocity_mps * (eta - eta_t)
        rows = np.nonzero(np.abs(x) <= 0.5 * l_s)[0]
        r_inst = np.sqrt(r_t * r_t + x[rows] ** 2)
        # delay of the echo in range samples, relative to the frame centre
        d = (r_inst - sc.r_center_m) / dr
        lo = np.maximum(np.ceil(d - half - 1e-9).astype(np.int64) + nr // 2, 0)
        carrier = np.exp(-1j * ((4.0 * np.pi / lam) * r_inst % (2.0 * np.pi)))
        for i, m in enumerate(rows):
            n0 = int(lo[i])
            n1 = min(n0 + sc.pulse_samples + 1, nr)
            u = ncol[n0:n1] - d[i]                       # samples from the pulse centre
            keep = (u >= -half - 1e-9) & (u < half - 1e-9)
            t = u[keep] / fs
            raw[m, n0:n1][keep] += np.exp(1j * np.pi * K * t * t) * carrier[i]
    if sc.noise_variance > 0.0:
        g = _rng(seed)
        s = np.sqrt(sc.noise_variance / 2.0)
        for m0 in range(0, na, 256):
            m1 = min(na, m0 + 256)
            nz = g.standard_normal((m1 - m0, nr, 2))
            raw[m0:m1] += s * (nz[..., 0] + 1j * nz[..., 1])
    return raw.astype(dtype)
