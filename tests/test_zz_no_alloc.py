"""The allocation-free entry point, for callers that cannot call cudaMalloc
while they process (a loop that must not stall the device, a process whose
device memory is already committed elsewhere): its scratch is a fixed array
inside the library. Checked through the C ABI against the plan-based two-pass
transform of the same size, on two calls in a row that share that array, and
against the oracle. Collected last, so a run that stops at the first failure
has already run every other test."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_noalloc_matches_the_plan_path_twice_in_a_row():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import oracle
    from paper_2609_32237_b200 import binding as B, inputs
    from gpu_util import run_fft, rel_l2, worst_rel_l2

    st = torch.cuda.current_stream().cuda_stream
    # two different sizes and directions back to back: the second call finds the
    # first call's scratch image and tables in the shared array
    for n, batch, direction, seed in ((1 << 16, 4, -1, 81), (1 << 15, 8, +1, 82), (1 << 16, 4, -1, 83)):
        x = inputs.gaussian_complex64((batch, n), seed)
        d = torch.from_numpy(x).cuda()
        got = torch.zeros_like(d)
        B.fft_execute_noalloc(n, batch, direction, d.data_ptr(), got.data_ptr(), st)
        torch.cuda.synchronize()
        ref = run_fft(d, n, batch, 1, n, direction, B.C64)            # existing entry point, same split
        assert rel_l2(got.cpu().numpy(), ref.cpu().numpy()) <= 1e-5
        want = oracle.fft_rows(x.astype(np.complex128), direction)
        worst, pooled = worst_rel_l2(got.cpu().numpy(), want)
        assert worst <= 1e-5 and pooled <= 1e-5
        # in place (the header allows in == out: the first pass has read the input before the second writes)
        same = d.clone()
        B.fft_execute_noalloc(n, batch, direction, same.data_ptr(), same.data_ptr(), st)
        torch.cuda.synchronize()
        assert bool((same == got).all())

    # sizes beyond the fixed scratch are refused with a clear status, not run
    big = torch.zeros(2 * B.NOALLOC_MAX_ELEMS, dtype=torch.complex64, device="cuda")
    with pytest.raises(B.B200FftError) as e:
        B.fft_execute_noalloc(1 << 16, 8, -1, big.data_ptr(), big.data_ptr(), st)
    assert e.value.status == 6
    with pytest.raises(B.B200FftError) as e:
        B.fft_execute_noalloc(1 << 20, 1, -1, big.data_ptr(), big.data_ptr(), st)
    assert e.value.status == 6
    with pytest.raises(B.B200FftError) as e:
        B.fft_execute_noalloc(1000, 1, -1, big.data_ptr(), big.data_ptr(), st)
    assert e.value.status == 2
