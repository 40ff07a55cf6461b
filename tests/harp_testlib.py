"""Shared helpers of the GPU parity tests: move seeded host arrays to the device,
call the library through its C ABI binding, bring results back as fp64."""
import numpy as np
import torch

import paper_2605_29843_b200 as harp
from paper_2605_29843_b200 import workloads as wl


def to_device(arr: np.ndarray, dtype: str) -> torch.Tensor:
    """arr: float32 array ('f32') or uint16 bf16 bit patterns ('bf16')."""
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).cuda()
    t = torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).cuda()
    return t.view(torch.bfloat16)


def to_host_f64(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.float32:
        return t.cpu().numpy().astype(np.float64)
    bits = t.view(torch.int16).cpu().numpy().view(np.uint16)
    return wl.bf16_bits_to_f64(bits)


def host_rows(x64: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64 test data once to the I/O dtype; returns the array handed to the GPU."""
    x32 = x64.astype(np.float32)
    return x32 if dtype == "f32" else wl.f32_to_bf16_bits(x32)


def promote(arr: np.ndarray, dtype: str) -> np.ndarray:
    return arr.astype(np.float64) if dtype == "f32" else wl.bf16_bits_to_f64(arr)


def gpu_apply(plan, host_arr: np.ndarray, dtype: str, transpose=False, kernel=harp.KERNEL_AUTO,
              guard_rows: int = 2):
    """Run harp_apply on a copy of host_arr placed between guard bands; returns
    (result fp64, guards_intact)."""
    n, d = host_arr.shape
    x = to_device(host_arr, dtype)
    canary = 1.0e4 if dtype == "f32" else 256.0
    buf = torch.full((n + 2 * guard_rows, d), canary, dtype=x.dtype, device="cuda")
    buf[guard_rows:guard_rows + n] = x
    view = buf[guard_rows:guard_rows + n]
    harp.harp_apply(plan, view.data_ptr(), n, harp.HARP_F32 if dtype == "f32" else harp.HARP_BF16,
                    transpose, torch.cuda.current_stream().cuda_stream, kernel)
    torch.cuda.synchronize()
    ok = bool((buf[:guard_rows] == canary).all() and (buf[guard_rows + n:] == canary).all())
    return to_host_f64(view), ok


TOL = {"f32": 1e-5, "bf16": 8e-3}
