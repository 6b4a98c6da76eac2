"""ctypes binding of libb200fft.so: argument marshalling only.

Every function here has the name and argument order of its C counterpart in
include/b200fft.h and raises B200FftError on a non-zero status. Device
pointers are plain integers (torch: tensor.data_ptr()); streams are
cudaStream_t handles as integers (torch: torch.cuda.current_stream().cuda_stream).
There is no CPU fallback: if the shared library is missing, importing fails.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libb200fft.so")

FORWARD, INVERSE = -1, 1
C64, C32H = 0, 1

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "ALIGNMENT", 4: "ALLOC", 5: "CUDA", 6: "WORKSPACE"}

EXPORTS = [
    "fft_plan_create", "fft_plan_workspace_bytes", "fft_plan_set_workspace", "fft_execute",
    "fft_execute_host", "fft_plan_destroy", "fft_plan_set_option", "fft_status_string",
    "b200fft_launch_count", "sar_rda_params_create", "sar_rda_workspace_bytes",
    "sar_rda_set_workspace", "sar_rda_form_image", "sar_rda_form_image_host", "sar_rda_run_step",
    "sar_rda_params_destroy", "fft_execute_noalloc", "sar_rda_set_option", "b200fft_tma_timeouts",
    "fft_execute_bfp", "sar_rda_shard_geometry_of", "sar_rda_shard_create", "sar_rda_shard_get_geometry",
    "sar_rda_shard_set_workspace", "sar_rda_shard_range_compress", "sar_rda_shard_azimuth", "sar_rda_shard_destroy",
]


class B200FftError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({STATUS_NAMES.get(status, '?')}: {status_string(status)})")


class SarRdaDesc(ctypes.Structure):
    _fields_ = [
        ("n_azimuth", ctypes.c_int64), ("n_range", ctypes.c_int64),
        ("carrier_hz", ctypes.c_double), ("bandwidth_hz", ctypes.c_double),
        ("fs_hz", ctypes.c_double), ("pulse_s", ctypes.c_double), ("prf_hz", ctypes.c_double),
        ("velocity_mps", ctypes.c_double), ("r_center_m", ctypes.c_double),
        ("intermediate_dtype", ctypes.c_int32), ("rcmc_taps", ctypes.c_int32),
    ]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_32237_b200.build` "
            "(nvcc, sm_100a). There is no CPU fallback.")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    L.fft_plan_create.argtypes = [ctypes.POINTER(vp), i64, i64, i64, i64, ci, ci]
    L.fft_plan_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    L.fft_plan_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    L.fft_execute.argtypes = [vp, vp, vp, vp]
    L.fft_execute_host.argtypes = [vp, vp, vp, vp, vp, vp]
    L.fft_plan_destroy.argtypes = [vp]
    L.fft_plan_set_option.argtypes = [vp, ctypes.c_char_p, i64]
    L.fft_status_string.argtypes = [ci]
    L.fft_status_string.restype = ctypes.c_char_p
    L.b200fft_launch_count.restype = i64
    L.sar_rda_params_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(SarRdaDesc)]
    L.sar_rda_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    L.sar_rda_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    L.sar_rda_form_image.argtypes = [vp, vp, vp, vp]
    L.sar_rda_form_image_host.argtypes = [vp, vp, vp, vp, vp, vp]
    L.sar_rda_run_step.argtypes = [vp, vp, vp, ci, vp]
    L.sar_rda_params_destroy.argtypes = [vp]
    L.fft_execute_noalloc.argtypes = [i64, i64, ci, vp, vp, vp]
    L.fft_execute_bfp.argtypes = [vp, vp, vp, vp, vp, vp]
    L.sar_rda_set_option.argtypes = [vp, ctypes.c_char_p, i64]
    L.sar_rda_shard_geometry_of.argtypes = [ctypes.POINTER(SarRdaDesc), ctypes.c_int32, ctypes.c_int32,
                                            ctypes.POINTER(SarShardGeometry)]
    L.sar_rda_shard_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(SarRdaDesc), ctypes.c_int32, ctypes.c_int32]
    L.sar_rda_shard_get_geometry.argtypes = [vp, ctypes.POINTER(SarShardGeometry)]
    L.sar_rda_shard_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    L.sar_rda_shard_range_compress.argtypes = [vp, vp, ctypes.POINTER(vp), vp]
    L.sar_rda_shard_azimuth.argtypes = [vp, vp, vp]
    L.sar_rda_shard_destroy.argtypes = [vp]
    return L


class SarShardGeometry(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int64) for name in (
        "first_pulse", "pulses", "first_bin", "bins", "halo_left", "halo_right", "strip_width", "strip_bytes",
        "workspace_bytes")]


_lib = _load()


def lib():
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise B200FftError(status, where)


def status_string(status: int) -> str:
    return _lib.fft_status_string(status).decode()


def tma_timeouts() -> int:
    return int(_lib.b200fft_tma_timeouts())


def launch_count() -> int:
    return int(_lib.b200fft_launch_count())


def fft_plan_create(n, batch, stride, dist, direction, storage_dtype) -> int:
    h = ctypes.c_void_p()
    _check(_lib.fft_plan_create(ctypes.byref(h), n, batch, stride, dist, direction, storage_dtype), "fft_plan_create")
    return h.value


def fft_plan_workspace_bytes(plan) -> int:
    b = ctypes.c_size_t()
    _check(_lib.fft_plan_workspace_bytes(plan, ctypes.byref(b)), "fft_plan_workspace_bytes")
    return int(b.value)


def fft_plan_set_workspace(plan, device_ptr, nbytes):
    _check(_lib.fft_plan_set_workspace(plan, device_ptr, nbytes), "fft_plan_set_workspace")


def fft_plan_set_option(plan, key: str, value: int):
    _check(_lib.fft_plan_set_option(plan, key.encode(), value), "fft_plan_set_option")


def fft_execute(plan, in_ptr, out_ptr, stream=0):
    _check(_lib.fft_execute(plan, in_ptr, out_ptr, stream), "fft_execute")


def fft_execute_host(plan, host_in, host_out, dev_in, dev_out, stream=0):
    _check(_lib.fft_execute_host(plan, host_in, host_out, dev_in, dev_out, stream), "fft_execute_host")


def fft_execute_noalloc(n, batch, direction, in_ptr, out_ptr, stream=0):
    """Two-pass transform of `batch` contiguous complex64 rows of n points that
    allocates nothing: scratch and tables live in a fixed array inside the
    library (n * batch <= NOALLOC_MAX_ELEMS). For callers that cannot call
    cudaMalloc while they process. Calls sharing the GPU must be ordered."""
    _check(_lib.fft_execute_noalloc(n, batch, direction, in_ptr, out_ptr, stream), "fft_execute_noalloc")


NOALLOC_MAX_ELEMS = 262144


def fft_execute_bfp(plan, in_ptr, in_exp_ptr, out_ptr, out_exp_ptr, stream=0):
    """Block-floating-point transform of fp16-stored rows: one int32 power-of-two exponent per
    transform on the way in (0 / None: all zero) and on the way out."""
    _check(_lib.fft_execute_bfp(plan, in_ptr, in_exp_ptr or None, out_ptr, out_exp_ptr, stream), "fft_execute_bfp")


def fft_plan_destroy(plan):
    _check(_lib.fft_plan_destroy(plan), "fft_plan_destroy")


def sar_rda_params_create(desc: SarRdaDesc) -> int:
    h = ctypes.c_void_p()
    _check(_lib.sar_rda_params_create(ctypes.byref(h), ctypes.byref(desc)), "sar_rda_params_create")
    return h.value


def sar_rda_workspace_bytes(params) -> int:
    b = ctypes.c_size_t()
    _check(_lib.sar_rda_workspace_bytes(params, ctypes.byref(b)), "sar_rda_workspace_bytes")
    return int(b.value)


def sar_rda_set_workspace(params, device_ptr, nbytes):
    _check(_lib.sar_rda_set_workspace(params, device_ptr, nbytes), "sar_rda_set_workspace")


def sar_rda_set_option(params, key: str, value: int):
    _check(_lib.sar_rda_set_option(params, key.encode(), value), "sar_rda_set_option")


def sar_rda_form_image(raw_ptr, params, out_ptr, stream=0):
    _check(_lib.sar_rda_form_image(raw_ptr, params, out_ptr, stream), "sar_rda_form_image")


def sar_rda_form_image_host(host_raw, params, host_out, dev_raw, dev_out, stream=0):
    _check(_lib.sar_rda_form_image_host(host_raw, params, host_out, dev_raw, dev_out, stream),
           "sar_rda_form_image_host")


def sar_rda_run_step(raw_ptr, params, out_ptr, step, stream=0):
    _check(_lib.sar_rda_run_step(raw_ptr, params, out_ptr, step, stream), "sar_rda_run_step")


def sar_rda_params_destroy(params):
    _check(_lib.sar_rda_params_destroy(params), "sar_rda_params_destroy")


def sar_rda_shard_geometry_of(desc: SarRdaDesc, rank: int, world: int) -> SarShardGeometry:
    g = SarShardGeometry()
    _check(_lib.sar_rda_shard_geometry_of(ctypes.byref(desc), rank, world, ctypes.byref(g)), "sar_rda_shard_geometry_of")
    return g


def sar_rda_shard_create(desc: SarRdaDesc, rank: int, world: int) -> int:
    h = ctypes.c_void_p()
    _check(_lib.sar_rda_shard_create(ctypes.byref(h), ctypes.byref(desc), rank, world), "sar_rda_shard_create")
    return h.value


def sar_rda_shard_get_geometry(shard) -> SarShardGeometry:
    g = SarShardGeometry()
    _check(_lib.sar_rda_shard_get_geometry(shard, ctypes.byref(g)), "sar_rda_shard_get_geometry")
    return g


def sar_rda_shard_set_workspace(shard, device_ptr, nbytes):
    _check(_lib.sar_rda_shard_set_workspace(shard, device_ptr, nbytes), "sar_rda_shard_set_workspace")


def sar_rda_shard_range_compress(shard, raw_rows_ptr, strip_ptrs, stream=0):
    arr = (ctypes.c_void_p * len(strip_ptrs))(*strip_ptrs)
    _check(_lib.sar_rda_shard_range_compress(shard, raw_rows_ptr, arr, stream), "sar_rda_shard_range_compress")


def sar_rda_shard_azimuth(shard, image_strip_ptr, stream=0):
    _check(_lib.sar_rda_shard_azimuth(shard, image_strip_ptr, stream), "sar_rda_shard_azimuth")


def sar_rda_shard_destroy(shard):
    _check(_lib.sar_rda_shard_destroy(shard), "sar_rda_shard_destroy")


def sar_desc_from_scene(scene, intermediate_dtype=C64) -> SarRdaDesc:
    """Marshal plain scene numbers (attribute names of inputs.SarScene) into the C struct."""
    return SarRdaDesc(
        n_azimuth=scene.n_azimuth, n_range=scene.n_range, carrier_hz=scene.carrier_hz,
        bandwidth_hz=scene.bandwidth_hz, fs_hz=scene.fs_hz, pulse_s=scene.pulse_s,
        prf_hz=scene.prf_hz, velocity_mps=scene.velocity_mps, r_center_m=scene.r_center_m,
        intermediate_dtype=intermediate_dtype, rcmc_taps=8)
