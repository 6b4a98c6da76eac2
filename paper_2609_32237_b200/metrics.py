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
