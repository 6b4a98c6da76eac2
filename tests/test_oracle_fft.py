"""Pins for the float64 DFT oracle: hand values, closed forms, invariants,
brute force on tiny inputs, and a library routine on special cases. None of
them re-types the oracle's own summation; a dropped term, a wrong sign or a
transposed index fails at least one."""
import cmath
import math

import numpy as np
import pytest

import oracle
from paper_2609_32237_b200 import inputs


def _rel(a, b):
    return np.linalg.norm(np.asarray(a) - np.asarray(b)) / np.linalg.norm(np.asarray(b))


# --- hand-evaluable values ---------------------------------------------------
def test_n1_identity():
    x = np.array([[3.0 - 2.0j]])
    assert oracle.fft_rows(x)[0, 0] == 3.0 - 2.0j
    assert oracle.fft_rows(x, +1)[0, 0] == 3.0 - 2.0j


def test_n2_sum_and_difference():
    x = np.array([[1.0 + 2.0j, 3.0 - 1.0j]])
    y = oracle.fft_rows(x)[0]
    assert y[0] == 4.0 + 1.0j and y[1] == -2.0 + 3.0j


def test_n4_shifted_impulse_fixes_the_sign():
    # delta at n=1: X[k] = exp(-2 pi i k / 4) = 1, -i, -1, +i for the forward transform
    x = np.array([[0, 1, 0, 0]], dtype=np.complex128)
    y = oracle.fft_rows(x)[0]
    np.testing.assert_allclose(y, [1, -1j, -1, 1j], atol=1e-15)
    # the inverse kernel has the other sign and carries 1/N
    z = oracle.fft_rows(x, +1)[0]
    np.testing.assert_allclose(z, np.array([1, 1j, -1, -1j]) / 4, atol=1e-15)


def test_n8_hand_values():
    # x[n] = n: X[0] = 28, X[k] = -4 + 4i cot(pi k / 8)  (arithmetic-progression closed form)
    x = np.arange(8, dtype=np.complex128)[None, :]
    y = oracle.fft_rows(x)[0]
    assert abs(y[0] - 28) < 1e-13
    for k in range(1, 8):
        assert abs(y[k] - (-4 + 4j / math.tan(math.pi * k / 8))) < 1e-12


@pytest.mark.parametrize("n", [1, 2, 4, 8, 64, 1024, 2048, 16384])
def test_impulse_gives_constant_and_ones_give_impulse(n):
    d = np.zeros((1, n), dtype=np.complex128)
    d[0, 0] = 1
    np.testing.assert_allclose(oracle.fft_rows(d)[0], np.ones(n), atol=1e-13)
    o = np.ones((1, n), dtype=np.complex128)
    y = oracle.fft_rows(o)[0]
    e = np.zeros(n, dtype=np.complex128)
    e[0] = n
    np.testing.assert_allclose(y, e, atol=1e-9 * n)


@pytest.mark.parametrize("n,m", [(8, 3), (1024, 17), (4096, 1000), (8192, 8191)])
def test_shifted_impulse_is_a_linear_phase(n, m):
    d = np.zeros((1, n), dtype=np.complex128)
    d[0, m] = 1
    y = oracle.fft_rows(d)[0]
    want = np.array([cmath.exp(-2j * cmath.pi * ((m * k) % n) / n) for k in range(n)])
    np.testing.assert_allclose(y, want, atol=1e-12)


@pytest.mark.parametrize("n,f0", [(16, 5), (1024, 300), (2048, 1), (16384, 12345)])
def test_single_tone_gives_a_delta(n, f0):
    t = np.arange(n)
    x = np.exp(2j * np.pi * ((f0 * t) % n) / n)[None, :]
    y = oracle.fft_rows(x)[0]
    want = np.zeros(n, dtype=np.complex128)
    want[f0] = n
    np.testing.assert_allclose(y, want, atol=1e-9 * n)


# --- brute force -------------------------------------------------------------
def _brute(x, sign):
    n = len(x)
    return [sum(x[m] * cmath.exp(sign * 2j * cmath.pi * m * k / n) for m in range(n))
            for k in range(n)]


@pytest.mark.parametrize("n", [3, 5, 8, 12, 32])
def test_direct_sum_against_python_brute_force(n):
    x = inputs.uniform_complex64((1, n), 11).astype(np.complex128)
    y = oracle.fft_rows(x, -1, method=1)[0]
    np.testing.assert_allclose(y, _brute(list(x[0]), -1), atol=1e-12)
    z = oracle.fft_rows(x, +1, method=1)[0]
    np.testing.assert_allclose(z, np.array(_brute(list(x[0]), +1)) / n, atol=1e-12)


def test_2d_against_brute_force_8x8():
    x = inputs.uniform_complex64((8, 8), 12).astype(np.complex128)
    y = oracle.fft2d(x)
    want = np.zeros((8, 8), dtype=np.complex128)
    for k1 in range(8):
        for k2 in range(8):
            want[k1, k2] = sum(x[a, b] * cmath.exp(-2j * cmath.pi * (a * k1 + b * k2) / 8)
                               for a in range(8) for b in range(8))
    np.testing.assert_allclose(y, want, atol=1e-11)


# --- the two methods agree, and agree with a library routine ------------------
@pytest.mark.parametrize("n", [64, 1024, 2048])
def test_recursion_equals_direct_sum(n):
    x = inputs.uniform_complex64((3, n), 13).astype(np.complex128)
    for d in (-1, +1):
        a = oracle.fft_rows(x, d, method=1)
        b = oracle.fft_rows(x, d, method=2)
        assert _rel(a, b) < 1e-14


@pytest.mark.parametrize("n", [1024, 4096, 16384])
def test_against_numpy_fft(n):
    x = inputs.gaussian_complex64((4, n), 14).astype(np.complex128)
    assert _rel(oracle.fft_rows(x, -1), np.fft.fft(x, axis=-1)) < 1e-14
    assert _rel(oracle.fft_rows(x, +1), np.fft.ifft(x, axis=-1)) < 1e-14


# --- invariants ---------------------------------------------------------------
@pytest.mark.parametrize("n", [1024, 4096])
def test_parseval_linearity_shift_roundtrip(n):
    x = inputs.uniform_complex64((2, n), 15).astype(np.complex128)
    X = oracle.fft_rows(x)
    # Parseval
    np.testing.assert_allclose((np.abs(X) ** 2).sum(-1), n * (np.abs(x) ** 2).sum(-1), rtol=1e-13)
    # linearity
    a, b = 0.3 - 1.1j, -2.0 + 0.5j
    lin = oracle.fft_rows((a * x[0] + b * x[1])[None, :])[0]
    assert _rel(lin, a * X[0] + b * X[1]) < 1e-14
    # circular shift by s multiplies bin k by exp(-2 pi i s k / n)
    s = 37
    Xs = oracle.fft_rows(np.roll(x[0], s)[None, :])[0]
    ph = np.exp(-2j * np.pi * ((s * np.arange(n)) % n) / n)
    assert _rel(Xs, X[0] * ph) < 1e-13
    # forward then inverse is the identity
    assert _rel(oracle.fft_rows(X, +1), x) < 1e-13
    # real input: conjugate symmetry
    r = oracle.fft_rows(x.real.astype(np.complex128))
    assert _rel(r[:, 1:], np.conj(r[:, :0:-1])) < 1e-13


# --- layouts -------------------------------------------------------------------
def test_columns_equal_transposed_rows():
    x = inputs.uniform_complex64((64, 48), 16).astype(np.complex128)
    cols = oracle.fft_cols(x)
    rows = oracle.fft_rows(np.ascontiguousarray(x.T)).T
    assert _rel(cols, rows) < 1e-14


def test_general_stride_and_dist():
    n, batch, stride, dist = 16, 3, 5, 1
    size = (batch - 1) * dist + (n - 1) * stride + 1
    buf = inputs.uniform_complex64((size,), 17).astype(np.complex128)
    out = oracle.fft_c2c(buf, n, batch, stride, dist, -1)
    for b in range(batch):
        want = np.fft.fft(buf[b * dist: b * dist + n * stride: stride])
        got = out[b * dist: b * dist + n * stride: stride]
        assert _rel(got, want) < 1e-14


def test_2d_is_rows_then_columns():
    x = inputs.uniform_complex64((32, 64), 18).astype(np.complex128)
    assert _rel(oracle.fft2d(x), np.fft.fft2(x)) < 1e-14


def test_unit_roots_octant_symmetry():
    n = 4096
    w = np.array([oracle.unit_root(j, n, -1) for j in range(n)])
    np.testing.assert_allclose(np.abs(w), 1.0, atol=2e-16)
    assert w[0] == 1 and w[n // 4] == -1j and w[n // 2] == -1 and w[3 * n // 4] == 1j
    assert abs(w[n // 8] - (1 - 1j) / math.sqrt(2)) < 2e-16
    np.testing.assert_allclose(w[1:], np.conj(w[:0:-1]), atol=1e-16)
    # forward and inverse roots are conjugates
    assert oracle.unit_root(5, 64, +1) == np.conj(oracle.unit_root(5, 64, -1))


# --- generators -----------------------------------------------------------------
def test_generators_are_seeded_and_in_range():
    a = inputs.uniform_complex64((256, 1024), 0)
    b = inputs.uniform_complex64((256, 1024), 0)
    assert a.dtype == np.complex64 and np.array_equal(a, b)
    v = a.view(np.float32)
    assert v.min() >= -1.0 and v.max() < 1.0
    assert abs(v.mean()) < 5e-3 and abs(v.var() - 1 / 3) < 5e-3
    g = inputs.gaussian_complex64((64, 4096), 1)
    gv = g.view(np.float32)
    assert abs(gv.mean()) < 1e-2 and abs(gv.std() - 1.0) < 1e-2
    assert not np.array_equal(inputs.gaussian_complex64((8, 8), 1), inputs.gaussian_complex64((8, 8), 2))
    h = inputs.to_half_storage(g)
    assert h.dtype == np.float16 and h.shape == g.shape + (2,)
    assert _rel(inputs.from_half_storage(h), g.astype(np.complex128)) < 1e-3
