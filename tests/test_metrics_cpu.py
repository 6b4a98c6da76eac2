"""The throughput arithmetic used by the bench, pinned to the numbers the paper prints."""
from paper_2609_32237_b200 import metrics
from conftest import read_golden


def test_eq1_ceilings_match_the_paper():
    g = read_golden("paper_eq1_ceilings.txt")
    bw = g["bandwidth_gbs"]
    for n in (4096, 8192, 16384):
        assert abs(metrics.single_pass_ceiling_gflops(n, bw, 0) - g[f"fp32_gflops_{n}"]) <= 0.6
        assert abs(metrics.single_pass_ceiling_gflops(n, bw, 1) - g[f"fp16_gflops_{n}"]) <= 1.0


def test_gflops_and_effective_bandwidth_are_consistent_with_the_paper_row():
    g = read_golden("paper_eq1_ceilings.txt")
    assert abs(metrics.gflops_to_gbs(g["row_gflops"], 4096, 0) - g["row_gbs"]) <= 1.0
    # a batch timed at exactly the ceiling reports the bandwidth it was derived from
    n, b = 8192, 2048
    secs = metrics.fft_bytes(n, b, 0) / (150e9)
    assert abs(metrics.fft_gflops(n, b, secs) - metrics.single_pass_ceiling_gflops(n, 150.0)) < 1e-6


def test_footprints():
    assert metrics.fft_bytes(4096, 32768, 0) == 2 * 1024 ** 3      # 1 GiB in + 1 GiB out
    assert metrics.fft_bytes(8192, 16384, 1) == 1024 ** 3
    assert metrics.sar_bytes(4096, 4096, 0) == 48 * 4096 * 4096
    assert metrics.sar_bytes(4096, 4096, 1) == 32 * 4096 * 4096


def test_issue_roof_arithmetic():
    # 148 multiprocessors x 4 schedulers x 1.965 GHz = 1.163e12 warp instructions per second
    assert abs(metrics.issue_roof_seconds(1.16328e12) - 1.0) < 1e-6
    # the fp16-storage transform of N = 8192 needs 213 us of issue slots against 164 us of HBM time
    t = metrics.issue_roof_seconds(metrics.NCU_WARP_INSTRUCTIONS["fft_rows_8192_b16384_c32h"])
    assert 2.1e-4 < t < 2.15e-4 and t > metrics.fft_bytes(8192, 16384, 1) / 6532.2e9
