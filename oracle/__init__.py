"""Python face of the CPU float64 oracle (oracle_fft.c, oracle_sar.c).

TEST INFRASTRUCTURE ONLY. Tests, the smoke check and the bench's CPU-baseline
leg may import this; the product package never does. It shares no code with
the CUDA path: the C sources here are compiled with gcc into liboracle.so and
called through ctypes with numpy complex128 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SOURCES = ["oracle_fft.c", "oracle_sar.c"]
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over independent transforms)."""
    srcs = [os.path.join(_HERE, s) for s in _SOURCES]
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in srcs)
    if stale:
        cmd = ["gcc", "-O2", "-std=gnu11", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", "-o", _LIB_PATH] + srcs + ["-lm"]
        subprocess.run(cmd, check=True)
    return _LIB_PATH


class SarParams(ctypes.Structure):
    _fields_ = [
        ("n_azimuth", ctypes.c_int64),
        ("n_range", ctypes.c_int64),
        ("pulse_samples", ctypes.c_int64),
        ("wavelength_m", ctypes.c_double),
        ("chirp_rate", ctypes.c_double),
        ("fs_hz", ctypes.c_double),
        ("prf_hz", ctypes.c_double),
        ("velocity_mps", ctypes.c_double),
        ("r_center_m", ctypes.c_double),
        ("rcmc_enabled", ctypes.c_int32),
        ("baseband_filter", ctypes.c_int32),
    ]


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB_PATH)
        dp = ctypes.POINTER(ctypes.c_double)
        i64 = ctypes.c_int64
        L.oracle_fft_c2c.argtypes = [i64, i64, i64, i64, ctypes.c_int, ctypes.c_int, dp, dp]
        L.oracle_fft2d.argtypes = [i64, i64, ctypes.c_int, dp, dp]
        L.oracle_unit_root.argtypes = [i64, i64, ctypes.c_int, dp]
        L.oracle_num_threads.restype = ctypes.c_int
        pp = ctypes.POINTER(SarParams)
        L.oracle_sar_matched_filter.argtypes = [pp, dp]
        for name in ("oracle_sar_range_compress", "oracle_sar_azimuth_fft", "oracle_sar_rcmc",
                     "oracle_sar_azimuth_filter", "oracle_sar_azimuth_ifft"):
            getattr(L, name).argtypes = [pp, dp, dp]
        L.oracle_sar_rda.argtypes = [pp, dp, dp, dp]
        L.oracle_sar_migration_bins.argtypes = [pp, i64, i64]
        L.oracle_sar_migration_bins.restype = ctypes.c_double
        L.oracle_sar_filter_phase.argtypes = [pp, i64, i64]
        L.oracle_sar_filter_phase.restype = ctypes.c_double
        L.oracle_sar_interp_weights.argtypes = [ctypes.c_double, dp]
        L.oracle_sar_interp_weights.restype = None
        _lib = L
    return _lib


def _dp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _c128(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.complex128)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def unit_root(j: int, n: int, sign: int) -> complex:
    out = np.zeros(2)
    if lib().oracle_unit_root(j, n, sign, _dp(out)):
        raise ValueError("bad unit_root arguments")
    return complex(out[0], out[1])


def fft_c2c(x, n: int, batch: int, stride: int, dist: int, direction: int,
            method: int = 0) -> np.ndarray:
    """Batched strided DFT over a flat complex buffer; element j of transform b
    at index b*dist + j*stride, same mapping in the returned buffer.
    direction -1 forward (unnormalised), +1 inverse (1/n).
    method 0: direct sum for n <= 1024, recursive radix-2 above; 1 / 2 force one."""
    xin = _c128(x).reshape(-1)
    need = (batch - 1) * dist + (n - 1) * stride + 1
    if xin.size < need:
        raise ValueError("input buffer too small")
    out = np.zeros_like(xin)
    rc = lib().oracle_fft_c2c(n, batch, stride, dist, direction, method, _dp(xin), _dp(out))
    if rc:
        raise ValueError(f"oracle_fft_c2c failed ({rc})")
    return out


def fft_rows(x: np.ndarray, direction: int = -1, method: int = 0) -> np.ndarray:
    """Transform along the last axis of a C-contiguous array."""
    x = _c128(x)
    n = x.shape[-1]
    b = x.size // n
    return fft_c2c(x, n, b, 1, n, direction, method).reshape(x.shape)


def fft_cols(x: np.ndarray, direction: int = -1) -> np.ndarray:
    """Transform along axis 0 of a row-major 2-D matrix, read in place (stride = width)."""
    x = _c128(x)
    rows, cols = x.shape
    return fft_c2c(x, rows, cols, cols, 1, direction).reshape(x.shape)


def fft2d(x: np.ndarray, direction: int = -1) -> np.ndarray:
    x = _c128(x)
    rows, cols = x.shape
    out = np.zeros_like(x)
    rc = lib().oracle_fft2d(rows, cols, direction, _dp(x), _dp(out))
    if rc:
        raise ValueError(f"oracle_fft2d failed ({rc})")
    return out


def sar_params(scene, rcmc_enabled: bool = True, baseband_filter: bool = True) -> SarParams:
    """Fill the oracle's parameter block from plain scene numbers (any object
    with the attribute names of paper_2609_32237_b200.inputs.SarScene)."""
    return SarParams(
        n_azimuth=scene.n_azimuth, n_range=scene.n_range,
        pulse_samples=int(round(scene.pulse_s * scene.fs_hz)),
        wavelength_m=299_792_458.0 / scene.carrier_hz,
        chirp_rate=scene.bandwidth_hz / scene.pulse_s,
        fs_hz=scene.fs_hz, prf_hz=scene.prf_hz, velocity_mps=scene.velocity_mps,
        r_center_m=scene.r_center_m,
        rcmc_enabled=int(bool(rcmc_enabled)), baseband_filter=int(bool(baseband_filter)))


def sar_matched_filter(p: SarParams) -> np.ndarray:
    H = np.zeros(p.n_range, dtype=np.complex128)
    rc = lib().oracle_sar_matched_filter(ctypes.byref(p), _dp(H))
    if rc:
        raise RuntimeError("oracle_sar_matched_filter failed")
    return H


def _sar_stage(name: str, p: SarParams, x: np.ndarray) -> np.ndarray:
    x = _c128(x)
    assert x.shape == (p.n_azimuth, p.n_range)
    out = np.zeros_like(x)
    rc = getattr(lib(), name)(ctypes.byref(p), _dp(x), _dp(out))
    if rc:
        raise RuntimeError(f"{name} failed ({rc})")
    return out


def sar_range_compress(p, raw):
    return _sar_stage("oracle_sar_range_compress", p, raw)


def sar_azimuth_fft(p, y):
    return _sar_stage("oracle_sar_azimuth_fft", p, y)


def sar_rcmc(p, S):
    return _sar_stage("oracle_sar_rcmc", p, S)


def sar_azimuth_filter(p, S1):
    return _sar_stage("oracle_sar_azimuth_filter", p, S1)


def sar_azimuth_ifft(p, S2):
    return _sar_stage("oracle_sar_azimuth_ifft", p, S2)


def sar_rda(p: SarParams, raw: np.ndarray, want_range_compressed: bool = False):
    raw = _c128(raw)
    assert raw.shape == (p.n_azimuth, p.n_range)
    img = np.zeros_like(raw)
    stage = np.zeros_like(raw) if want_range_compressed else None
    rc = lib().oracle_sar_rda(ctypes.byref(p), _dp(raw), _dp(img),
                              _dp(stage) if stage is not None else None)
    if rc:
        raise RuntimeError(f"oracle_sar_rda failed ({rc})")
    return (img, stage) if want_range_compressed else img


def sar_migration_bins(p: SarParams, k: int, n: int) -> float:
    return float(lib().oracle_sar_migration_bins(ctypes.byref(p), k, n))


def sar_filter_phase(p: SarParams, k: int, n: int) -> float:
    return float(lib().oracle_sar_filter_phase(ctypes.byref(p), k, n))


def sar_interp_weights(mu: float) -> np.ndarray:
    w = np.zeros(8)
    lib().oracle_sar_interp_weights(mu, _dp(w))
    return w
