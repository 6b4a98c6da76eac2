"""GPU parity of the block-floating-point row transform (fp16 storage, one power-of-two
exponent per transform) against the float64 oracle: the dequantised result must match the
plain DFT of the dequantised input within the fp16 tolerance, the stored mantissas must use
the range [2^14, 2^15), and coherent inputs that overflow the plain fp16 plan must survive."""
import numpy as np
import pytest

import oracle
from paper_2609_32237_b200 import inputs
from gpu_util import have_gpu, rel_l2, worst_rel_l2, to_device_half, half_to_c128, run_fft

pytestmark = pytest.mark.gpu
FWD, INV = -1, 1
C32H = 1
TOL16 = 5e-3


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not have_gpu():
        pytest.skip("no CUDA device")


def _bfp(h, n, batch, direction, in_exp=None, inplace=False):
    import torch
    from paper_2609_32237_b200 import binding as B
    d = to_device_half(h)
    out = d if inplace else torch.zeros_like(d)
    e_out = torch.full((batch,), 12345, dtype=torch.int32, device="cuda")
    e_in = None if in_exp is None else torch.from_numpy(np.asarray(in_exp, dtype=np.int32)).cuda()
    plan = B.fft_plan_create(n, batch, 1, n, direction, C32H)
    try:
        B.fft_execute_bfp(plan, d.data_ptr(), 0 if e_in is None else e_in.data_ptr(), out.data_ptr(),
                          e_out.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
    finally:
        B.fft_plan_destroy(plan)
    return out.cpu().numpy(), e_out.cpu().numpy()


def _dequant(stored, exps):
    return inputs.from_half_storage(stored) * np.exp2(exps.astype(np.float64))[:, None]


def _mantissa_range_ok(stored):
    m = np.abs(stored.astype(np.float64)).reshape(stored.shape[0], -1).max(axis=1)
    return np.all((m >= 16384.0) & (m <= 32768.0))      # 32768 itself only by rounding up from just below


@pytest.mark.parametrize("n", [1024, 2048, 4096, 8192, 16384])
@pytest.mark.parametrize("direction", [FWD, INV])
def test_noise_rows_every_size(n, direction):
    batch = 7
    x = inputs.gaussian_complex64((batch, n), 500 + n) * np.float32(3.0)
    h = inputs.to_half_storage(x)
    e_in = np.array([0, 3, -5, 11, 0, -20, 7], dtype=np.int32)
    stored, e_out = _bfp(h, n, batch, direction, e_in)
    x_true = inputs.from_half_storage(h) * np.exp2(e_in.astype(np.float64))[:, None]
    want = oracle.fft_rows(x_true, direction)
    got = _dequant(stored, e_out)
    assert max(worst_rel_l2(got, want)) <= TOL16
    assert _mantissa_range_ok(stored)
    # without input exponents, and in place
    stored2, e2 = _bfp(h, n, batch, direction, None, inplace=True)
    assert np.array_equal(stored2.view(np.uint16), stored.view(np.uint16))
    assert np.array_equal(e2, e_out - e_in)


def test_coherent_rows_overflow_the_plain_plan_but_not_this_one():
    """A strong tone: the spectrum peak is N times the amplitude, far beyond 65504."""
    n, batch = 8192, 5
    k0 = np.array([0, 1, 37, 4095, 8191])
    t = np.arange(n)
    x = (100.0 * np.exp(2j * np.pi * k0[:, None] * t[None, :] / n)).astype(np.complex64)
    x += inputs.gaussian_complex64((batch, n), 9) * np.float32(0.1)
    h = inputs.to_half_storage(x)
    plain = half_to_c128(run_fft(to_device_half(h), n, batch, 1, n, FWD, C32H))
    assert not np.isfinite(np.abs(plain)).all()                   # the point of the exercise
    stored, e_out = _bfp(h, n, batch, FWD)
    got = _dequant(stored, e_out)
    want = oracle.fft_rows(inputs.from_half_storage(h), FWD)
    assert np.isfinite(np.abs(got)).all()
    assert max(worst_rel_l2(got, want)) <= TOL16
    assert _mantissa_range_ok(stored)
    assert np.all(e_out >= 4)                                      # 100 * 8192 / 2^15 = 25: at least 2^4
    peak = np.argmax(np.abs(got), axis=1)
    assert np.array_equal(peak, k0)


def test_forward_then_inverse_round_trip_carries_the_exponents():
    n, batch = 4096, 9
    x = inputs.gaussian_complex64((batch, n), 77) * np.float32(50.0)
    h = inputs.to_half_storage(x)
    s1, e1 = _bfp(h, n, batch, FWD)
    s2, e2 = _bfp(s1, n, batch, INV, e1)
    back = _dequant(s2, e2)
    assert rel_l2(back, inputs.from_half_storage(h)) <= TOL16
    assert _mantissa_range_ok(s2)


def test_zero_rows_and_error_paths():
    import torch
    from paper_2609_32237_b200 import binding as B
    n, batch = 1024, 3
    h = np.zeros((batch, n, 2), dtype=np.float16)
    h[1, 5, 0] = 1.0                                               # one impulse row between two zero rows
    stored, e_out = _bfp(h, n, batch, FWD)
    assert e_out[0] == 0 and e_out[2] == 0 and np.all(stored[0] == 0) and np.all(stored[2] == 0)
    assert e_out[1] == -14                                         # |X| = 1 everywhere: stored 2^14
    assert np.all(np.abs(np.abs(half_to_c128(torch.from_numpy(stored[1]))) - 16384.0) <= 16.0)   # fp16 spacing is 8 here
    d = to_device_half(h)
    e = torch.zeros(batch, dtype=torch.int32, device="cuda")
    p64 = B.fft_plan_create(n, batch, 1, n, FWD, 0)                # complex64 storage: not this call
    try:
        with pytest.raises(B.B200FftError) as err:
            B.fft_execute_bfp(p64, d.data_ptr(), 0, d.data_ptr(), e.data_ptr(), 0)
        assert err.value.status == 2
    finally:
        B.fft_plan_destroy(p64)
    p512 = B.fft_plan_create(512, batch, 1, 512, FWD, C32H)        # below the supported sizes
    try:
        with pytest.raises(B.B200FftError) as err:
            B.fft_execute_bfp(p512, d.data_ptr(), 0, d.data_ptr(), e.data_ptr(), 0)
        assert err.value.status == 2
    finally:
        B.fft_plan_destroy(p512)
    p = B.fft_plan_create(n, batch, 1, n, FWD, C32H)
    try:
        with pytest.raises(B.B200FftError) as err:
            B.fft_execute_bfp(p, d.data_ptr(), 0, d.data_ptr(), 0, 0)      # no place for the exponents
        assert err.value.status == 1
    finally:
        B.fft_plan_destroy(p)
