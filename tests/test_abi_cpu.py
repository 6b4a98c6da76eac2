"""Host-only checks of the C-ABI library: it loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2609_32237_b200 import build
    build.build()
    from paper_2609_32237_b200 import binding
    return binding


def test_header_symbols_are_exported(B):
    hdr = open(os.path.join(ROOT, "include", "b200fft.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b((?:fft|sar_rda|b200fft)_[a-z_0-9]+)\s*\(", hdr))
    assert names, "no prototypes found"
    assert names == set(B.EXPORTS)
    for n in names:
        assert hasattr(B.lib(), n), n


def test_status_strings(B):
    assert B.status_string(0) == "ok"
    for s in range(1, 7):
        assert B.status_string(s) not in ("ok", "unknown status")
    assert B.status_string(99) == "unknown status"


def test_bad_arguments_are_rejected_on_the_host(B):
    L = B.lib()
    h = ctypes.c_void_p()
    assert L.fft_plan_create(None, 1024, 1, 1, 1024, -1, 0) == 1
    assert L.fft_plan_create(ctypes.byref(h), 0, 1, 1, 1024, -1, 0) == 1
    assert L.fft_plan_create(ctypes.byref(h), 1024, 0, 1, 1024, -1, 0) == 1
    assert L.fft_plan_create(ctypes.byref(h), 1024, 1, 1, 1024, 0, 0) == 1       # direction
    assert L.fft_plan_create(ctypes.byref(h), 1024, 1, 1, 1024, -1, 7) == 1      # dtype
    assert L.fft_plan_create(ctypes.byref(h), 1000, 1, 1, 1000, -1, 0) == 2      # not a power of two
    assert L.fft_plan_create(ctypes.byref(h), 4, 1, 1, 4, -1, 0) == 2            # too small
    assert L.fft_plan_create(ctypes.byref(h), 1 << 21, 1, 1, 1 << 21, -1, 0) == 2
    assert L.fft_plan_create(ctypes.byref(h), 1024, 4, 3, 7, -1, 0) == 2         # layout class
    assert L.fft_plan_create(ctypes.byref(h), 1024, 4, 1, 1025, -1, 0) == 3      # odd dist
    assert L.fft_plan_create(ctypes.byref(h), 1024, 3, 4, 1, -1, 0) == 3         # odd column count
    assert h.value is None
    assert L.fft_execute(None, None, None, None) == 1
    assert L.fft_plan_destroy(None) == 1
    assert L.fft_execute_bfp(None, None, None, None, None, None) == 1
    assert L.fft_plan_set_option(None, b"staged", 1) == 1
    assert L.fft_execute_noalloc(4096, 1 << 20, -1, None, None, None) != 0     # beyond the fixed scratch, or null
    assert L.sar_rda_params_create(None, None) == 1
    d = B.SarRdaDesc(n_azimuth=4096, n_range=4096, carrier_hz=9.6e9, bandwidth_hz=1e8, fs_hz=1.2e8,
                     pulse_s=1e-5, prf_hz=1000.0, velocity_mps=200.0, r_center_m=1e4,
                     intermediate_dtype=0, rcmc_taps=6)
    assert L.sar_rda_params_create(ctypes.byref(h), ctypes.byref(d)) == 2        # only 8 taps
    d.rcmc_taps = 8
    d.intermediate_dtype = 5
    assert L.sar_rda_params_create(ctypes.byref(h), ctypes.byref(d)) == 1
    d.intermediate_dtype = 0
    d.velocity_mps = 1e-3                                                          # D would not be real
    assert L.sar_rda_params_create(ctypes.byref(h), ctypes.byref(d)) == 1


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_32237_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "liboracle" not in text, f
