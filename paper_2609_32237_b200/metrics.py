"""Throughput bookkeeping (host arithmetic only; none of the method's steps).

The paper counts 5 N log2 N floating-point operations per complex transform
and reports effective bandwidth as bytes in plus bytes out over time (Section
"Platform and Methodology", "Throughput"); a single pass moves 16 bytes per
point in fp32 storage and 8 in fp16 storage, which gives the ceiling of Eq. 1.
"""
from __future__ import annotations

import math

BYTES_PER_POINT = {0: 16, 1: 8}        # storage dtype -> bytes in + bytes out per point

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures
# summarised under profiles/ (None until a capture exists for that kernel)
NCU_TRAFFIC_BYTES = {"fft_rows_4096_c64": 2095526000}


# smsp__inst_executed.sum (warp instructions) per launch or per image from the same captures, for the
# workloads whose roof is instruction issue rather than HBM
NCU_WARP_INSTRUCTIONS = {
    "fft_rows_8192_b16384_c32h": 247463936,
    "fft_rows_16384_b8192_c32h": 266299384,
    "sar_4096x4096_fp32": 54689792 + 27472854 + 59949056 + 27695506,
    "sar_4096x4096_fp16": 55210000 + 28980000 + 66140000 + 27700000,
}


def issue_roof_seconds(warp_instructions: float, sms: int = 148, schedulers_per_sm: int = 4, sm_mhz: float = 1965.0) -> float:
    """Shortest time in which one GPU can issue that many warp instructions: every scheduler of every
    multiprocessor issues at most one per cycle."""
    return warp_instructions / (sms * schedulers_per_sm * sm_mhz * 1e6)


def fft_flops(n: int, batch: int = 1) -> float:
    return 5.0 * n * math.log2(n) * batch


def fft_bytes(n: int, batch: int, storage_dtype: int = 0) -> int:
    return BYTES_PER_POINT[storage_dtype] * n * batch


def fft_gflops(n: int, batch: int, seconds: float) -> float:
    return fft_flops(n, batch) / seconds / 1e9


def single_pass_ceiling_gflops(n: int, bandwidth_gbs: float, storage_dtype: int = 0) -> float:
    """Eq. 1: bandwidth * 5 log2 N / bytes per point."""
    return bandwidth_gbs * 5.0 * math.log2(n) / BYTES_PER_POINT[storage_dtype]


def gflops_to_gbs(gflops: float, n: int, storage_dtype: int = 0) -> float:
    return gflops * BYTES_PER_POINT[storage_dtype] / (5.0 * math.log2(n))


def sar_bytes(n_azimuth: int, n_range: int, intermediate_dtype: int = 0) -> int:
    """Three passes: raw fp32 in, two intermediate images written and read, fp32 image out."""
    inter = 8 if intermediate_dtype == 0 else 4
    return n_azimuth * n_range * (8 + inter + inter + inter + inter + 8)
