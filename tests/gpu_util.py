"""Helpers for the GPU parity tests: move numpy arrays through torch device
memory and call the C ABI. torch is used for memory and streams only."""
import numpy as np


def have_gpu():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def rel_l2(got, want):
    got = np.asarray(got, dtype=np.complex128)
    want = np.asarray(want, dtype=np.complex128)
    return float(np.linalg.norm(got - want) / np.linalg.norm(want))


def worst_rel_l2(got, want):
    """Worst single transform (last axis) and pooled relative L2 error."""
    got = np.asarray(got, dtype=np.complex128).reshape(-1, got.shape[-1])
    want = np.asarray(want, dtype=np.complex128).reshape(-1, want.shape[-1])
    per = np.linalg.norm(got - want, axis=1) / np.linalg.norm(want, axis=1)
    return float(per.max()), rel_l2(got, want)


def to_device_c64(x):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.complex64)).cuda()


def to_device_half(h):
    """h: float16 array (..., 2)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(h)).cuda()


def run_fft(x_dev, n, batch, stride, dist, direction, dtype, inplace=False, options=None, out_dev=None):
    """Execute one plan on a device tensor; returns the output tensor."""
    import torch
    from paper_2609_32237_b200 import binding as B
    plan = B.fft_plan_create(n, batch, stride, dist, direction, dtype)
    try:
        for k, v in (options or {}).items():
            B.fft_plan_set_option(plan, k, v)
        ws = None
        need = B.fft_plan_workspace_bytes(plan)
        if need:
            ws = torch.empty(need, dtype=torch.uint8, device="cuda")
            B.fft_plan_set_workspace(plan, ws.data_ptr(), need)
        out = x_dev if inplace else (out_dev if out_dev is not None else torch.zeros_like(x_dev))
        B.fft_execute(plan, x_dev.data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        return out
    finally:
        B.fft_plan_destroy(plan)


def half_to_c128(t):
    """device/host float16 tensor (..., 2) -> numpy complex128."""
    a = t.cpu().numpy().astype(np.float64)
    return a[..., 0] + 1j * a[..., 1]
