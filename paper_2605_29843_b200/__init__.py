"""B200-native HARP apply: thin ctypes binding over libharp.so.

The functions here carry the same names as the C ABI in ``include/harp.h`` and do
argument marshalling only; every step of the path runs in the CUDA library.  There is
no CPU fallback: if the library is missing or fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libharp.so")

HARP_F32, HARP_BF16 = 0, 1
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_FAST, KERNEL_SPLIT, KERNEL_TMEM = 0, 1, 2, 3, 4
HARP_OK = 0
HARP_ERR_UNSUPPORTED = 8

_lib: Optional[ctypes.CDLL] = None


class HarpError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = int(status)
        super().__init__(f"{what}: {status_string(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Load libharp.so (built in-tree by ``paper_2605_29843_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: run `python -m paper_2605_29843_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
        L.harp_plan_create.restype = ctypes.c_int
        L.harp_plan_create.argtypes = [ctypes.POINTER(vp), i64, i32, vp, vp, vp, ctypes.POINTER(vp)]
        L.harp_greedy_schedule.restype = i32
        L.harp_greedy_schedule.argtypes = [i64, i32, i32, vp, i32]
        L.harp_theta_params_per_block.restype = i32
        L.harp_theta_params_per_block.argtypes = [i32]
        L.harp_blocks_from_theta.restype = ctypes.c_int
        L.harp_blocks_from_theta.argtypes = [i32, i64, vp, vp, vp, vp, vp]
        L.harp_grad_theta.restype = ctypes.c_int
        L.harp_grad_theta.argtypes = [i32, i64, vp, vp, vp, vp]
        L.harp_plan_create_from_theta.restype = ctypes.c_int
        L.harp_plan_create_from_theta.argtypes = [ctypes.POINTER(vp), i64, i32, vp, vp, vp, vp, vp, vp, vp]
        L.harp_plan_create_kronecker.restype = ctypes.c_int
        L.harp_plan_create_kronecker.argtypes = [ctypes.POINTER(vp), i64, i32, vp, ctypes.POINTER(vp), i32, vp, vp, vp]
        L.harp_plan_destroy.restype = None
        L.harp_plan_destroy.argtypes = [vp]
        L.harp_plan_dim.restype = i64
        L.harp_plan_dim.argtypes = [vp]
        L.harp_apply.restype = ctypes.c_int
        L.harp_apply.argtypes = [vp, vp, i64, ctypes.c_int, ctypes.c_int, vp]
        L.harp_apply_ex.restype = ctypes.c_int
        L.harp_apply_ex.argtypes = [vp, vp, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp]
        L.harp_apply_passes.restype = ctypes.c_int
        L.harp_apply_passes.argtypes = [ctypes.POINTER(vp), i32, vp, i64, ctypes.c_int, ctypes.c_int, vp]
        L.harp_apply_two_sided.restype = ctypes.c_int
        L.harp_apply_two_sided.argtypes = [vp, ctypes.c_int, vp, vp, vp, vp]
        L.harp_two_sided_scratch_bytes.restype = i64
        L.harp_two_sided_scratch_bytes.argtypes = [vp, vp, ctypes.c_int]
        L.harp_apply_two_sided_static.restype = ctypes.c_int
        L.harp_apply_two_sided_static.argtypes = [vp, ctypes.c_int, vp, vp, vp]
        L.harp_two_sided_static_capacity_bytes.restype = i64
        L.harp_two_sided_static_capacity_bytes.argtypes = []
        L.harp_grad_blocks.restype = ctypes.c_int
        L.harp_grad_blocks.argtypes = [vp, vp, vp, i64, ctypes.c_int, vp, ctypes.c_int, vp]
        L.harp_plan_n_params.restype = i64
        L.harp_plan_n_params.argtypes = [vp]
        L.harp_weight_incoherence.restype = ctypes.c_int
        L.harp_weight_incoherence.argtypes = [vp, i64, i64, ctypes.c_int, vp, vp]
        L.harp_offblock_energy.restype = ctypes.c_int
        L.harp_offblock_energy.argtypes = [vp, i64, i64, ctypes.c_int, vp, vp]
        L.harp_diag_weighted_error.restype = ctypes.c_int
        L.harp_diag_weighted_error.argtypes = [vp, vp, i64, i64, ctypes.c_int, vp, ctypes.c_int, vp, vp]
        L.harp_apply_host.restype = ctypes.c_int
        L.harp_apply_host.argtypes = [vp, vp, i64, ctypes.c_int, ctypes.c_int]
        L.harp_blocks_from_theta_device.restype = ctypes.c_int
        L.harp_blocks_from_theta_device.argtypes = [i32, i64, vp, vp, vp, vp, vp, vp]
        L.harp_theta_device_max_radix.restype = i32
        L.harp_theta_device_max_radix.argtypes = []
        L.harp_plan_error_word.restype = i32
        L.harp_plan_error_word.argtypes = [vp]
        L.harp_launch_count.restype = i64
        L.harp_launch_count.argtypes = []
        L.harp_status_string.restype = ctypes.c_char_p
        L.harp_status_string.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().harp_status_string(int(status)).decode()


def _debug_timing(fn_name: str, reset: bool):
    L = lib()
    fn = getattr(L, fn_name)
    fn.restype = ctypes.c_int32
    fn.argtypes = [ctypes.c_void_p, ctypes.c_int32]
    out = (ctypes.c_int64 * 16)()
    if fn(out, 1 if reset else 0) != 0:
        raise HarpError(10, fn_name)
    return list(out)


def harp_debug_tm_timing(reset: bool = True):
    return _debug_timing("harp_debug_tm_timing", reset)


def harp_debug_fast_timing(reset: bool = True):
    return _debug_timing("harp_debug_fast_timing", reset)


def harp_plan_error_word(plan) -> int:
    return int(lib().harp_plan_error_word(plan.handle if hasattr(plan, "handle") else plan))


def harp_launch_count() -> int:
    return int(lib().harp_launch_count())


class Plan:
    """Owner of a ``harp_plan_t*``; destroyed with the object."""

    def __init__(self, handle: int, d: int):
        self.handle = handle
        self.d = d

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and _lib is not None:
            _lib.harp_plan_destroy(h)


def harp_plan_create_status(d: int, radices: Sequence[int], perm, signs, blocks):
    """Raw call: returns (status, Plan or None).  Arrays are host numpy arrays."""
    L = lib()
    rad = np.ascontiguousarray(radices, dtype=np.int32)
    pm = None if perm is None else np.ascontiguousarray(perm, dtype=np.int32)
    sg = None if signs is None else np.ascontiguousarray(signs, dtype=np.int8)
    blks = [np.ascontiguousarray(b, dtype=np.float32) for b in blocks] if blocks is not None else None
    if blks is not None:
        arr = (ctypes.c_void_p * max(1, len(blks)))(*[b.ctypes.data for b in blks])
    else:
        arr = None
    out = ctypes.c_void_p()
    st = L.harp_plan_create(ctypes.byref(out), int(d), len(rad), rad.ctypes.data,
                            None if pm is None else pm.ctypes.data,
                            None if sg is None else sg.ctypes.data, arr)
    if st != HARP_OK:
        return st, None
    return st, Plan(out.value, int(d))


def harp_plan_create(d: int, radices: Sequence[int], perm=None, signs=None, blocks=None) -> Plan:
    st, plan = harp_plan_create_status(d, radices, perm, signs, blocks)
    if st != HARP_OK:
        raise HarpError(st, "harp_plan_create")
    return plan


def harp_greedy_schedule(d: int, b_base: int = 8, b_max: int = 8):
    buf = (ctypes.c_int32 * 64)()
    n = lib().harp_greedy_schedule(int(d), int(b_base), int(b_max), buf, 64)
    if n < 0:
        raise HarpError(3, "harp_greedy_schedule")
    return [int(buf[i]) for i in range(n)]


def harp_theta_params_per_block(b: int) -> int:
    return int(lib().harp_theta_params_per_block(int(b)))


def _ptr_array(arrs):
    if arrs is None:
        return None, None
    keep = [None if a is None else np.ascontiguousarray(a) for a in arrs]
    return (ctypes.c_void_p * len(keep))(*[None if a is None else a.ctypes.data for a in keep]), keep


def harp_blocks_from_theta(b: int, theta=None, theta_q=None, scales=None, mixer=None) -> np.ndarray:
    """Host-only: blocks[n_blocks, b, b] (float32) from per-block parameters."""
    npar = harp_theta_params_per_block(b)
    th = None if theta is None else np.ascontiguousarray(theta, dtype=np.float32).reshape(-1, npar)
    tq = None if theta_q is None else np.ascontiguousarray(theta_q, dtype=np.int8).reshape(-1, npar)
    sc = None if scales is None else np.ascontiguousarray(scales, dtype=np.float32)
    mx = None if mixer is None else np.ascontiguousarray(mixer, dtype=np.float32)
    n = (th if th is not None else tq).shape[0]
    out = np.empty((n, b, b), dtype=np.float32)
    st = lib().harp_blocks_from_theta(int(b), n, None if th is None else th.ctypes.data,
                                      None if tq is None else tq.ctypes.data, None if sc is None else sc.ctypes.data,
                                      None if mx is None else mx.ctypes.data, out.ctypes.data)
    if st != HARP_OK:
        raise HarpError(st, "harp_blocks_from_theta")
    return out


def harp_grad_theta(b: int, theta, grad_blocks, mixer=None) -> np.ndarray:
    """Host-only: dL/dtheta[n_blocks, n_par] (float32) from dL/dB[n_blocks, b, b]."""
    npar = harp_theta_params_per_block(b)
    th = np.ascontiguousarray(theta, dtype=np.float32).reshape(-1, npar)
    gb = np.ascontiguousarray(grad_blocks, dtype=np.float32).reshape(-1, b, b)
    if gb.shape[0] != th.shape[0]:
        raise ValueError("theta and grad_blocks disagree on the number of blocks")
    mx = None if mixer is None else np.ascontiguousarray(mixer, dtype=np.float32)
    out = np.empty_like(th)
    st = lib().harp_grad_theta(int(b), th.shape[0], th.ctypes.data, None if mx is None else mx.ctypes.data,
                               gb.ctypes.data, out.ctypes.data)
    if st != HARP_OK:
        raise HarpError(st, "harp_grad_theta")
    return out


def harp_theta_device_max_radix() -> int:
    return int(lib().harp_theta_device_max_radix())


def harp_blocks_from_theta_device(b: int, n_blocks: int, theta_ptr: int, theta_q_ptr: int, scales_ptr: int, mixer_ptr: int,
                                  out_ptr: int, stream: int = 0) -> None:
    """Device pointers in, block kernels float[n_blocks][b][b] out (device)."""
    st = lib().harp_blocks_from_theta_device(int(b), int(n_blocks), theta_ptr or None, theta_q_ptr or None,
                                             scales_ptr or None, mixer_ptr or None, out_ptr, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_blocks_from_theta_device")


def harp_plan_create_from_theta(d: int, radices: Sequence[int], perm=None, signs=None, theta=None, theta_q=None,
                                scales=None, mixers=None) -> Plan:
    rad = np.ascontiguousarray(radices, dtype=np.int32)
    pm = None if perm is None else np.ascontiguousarray(perm, dtype=np.int32)
    sg = None if signs is None else np.ascontiguousarray(signs, dtype=np.int8)
    th, k1 = _ptr_array(None if theta is None else [np.asarray(a, dtype=np.float32) for a in theta])
    tq, k2 = _ptr_array(None if theta_q is None else [np.asarray(a, dtype=np.int8) for a in theta_q])
    sc, k3 = _ptr_array(None if scales is None else [np.asarray(a, dtype=np.float32) for a in scales])
    mx, k4 = _ptr_array(None if mixers is None else [None if a is None else np.asarray(a, dtype=np.float32) for a in mixers])
    out = ctypes.c_void_p()
    st = lib().harp_plan_create_from_theta(ctypes.byref(out), int(d), len(rad), rad.ctypes.data,
                                           None if pm is None else pm.ctypes.data, None if sg is None else sg.ctypes.data,
                                           th, tq, sc, mx)
    if st != HARP_OK:
        raise HarpError(st, "harp_plan_create_from_theta")
    return Plan(out.value, int(d))


def harp_plan_create_kronecker(n2: int, radices: Sequence[int], blocks_n2, K: int, hk, perm=None, signs=None) -> Plan:
    rad = np.ascontiguousarray(radices, dtype=np.int32)
    blks = [np.ascontiguousarray(b, dtype=np.float32) for b in blocks_n2]
    arr = (ctypes.c_void_p * len(blks))(*[b.ctypes.data for b in blks])
    h = np.ascontiguousarray(hk, dtype=np.float32)
    pm = None if perm is None else np.ascontiguousarray(perm, dtype=np.int32)
    sg = None if signs is None else np.ascontiguousarray(signs, dtype=np.int8)
    out = ctypes.c_void_p()
    st = lib().harp_plan_create_kronecker(ctypes.byref(out), int(n2), len(rad), rad.ctypes.data, arr, int(K), h.ctypes.data,
                                          None if pm is None else pm.ctypes.data, None if sg is None else sg.ctypes.data)
    if st != HARP_OK:
        raise HarpError(st, "harp_plan_create_kronecker")
    return Plan(out.value, int(K) * int(n2))


def plan_from_spec(spec) -> Plan:
    """Plan from a ``workloads.PlanSpec``-like object (d, radices, perm, signs, blocks)."""
    return harp_plan_create(spec.d, spec.radices, spec.perm, spec.signs, spec.blocks)


def harp_plan_dim(plan: Plan) -> int:
    return int(lib().harp_plan_dim(plan.handle))


def harp_apply(plan: Plan, x_ptr: int, n_rows: int, dtype: int, transpose: bool = False,
               stream: int = 0, kernel: int = KERNEL_AUTO) -> None:
    """x_ptr: device address of n_rows x d elements, transformed in place on ``stream``."""
    st = lib().harp_apply_ex(plan.handle, x_ptr, int(n_rows), int(dtype), 1 if transpose else 0,
                             int(kernel), stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_apply")


def harp_apply_passes(plans, x_ptr: int, n_rows: int, dtype: int, transpose: bool = False, stream: int = 0) -> None:
    """Several passes: x <- x Q_0 Q_1 ... (or the transposes in the opposite order)."""
    arr = (ctypes.c_void_p * len(plans))(*[p.handle for p in plans])
    st = lib().harp_apply_passes(arr, len(plans), x_ptr, int(n_rows), int(dtype), 1 if transpose else 0, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_apply_passes")


def harp_apply_two_sided(w_ptr: int, dtype: int, plan_out: Plan, plan_in: Plan,
                         scratch_ptr: int = 0, stream: int = 0) -> None:
    st = lib().harp_apply_two_sided(w_ptr, int(dtype), plan_out.handle, plan_in.handle,
                                    scratch_ptr or None, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_apply_two_sided")


def harp_apply_two_sided_static(w_ptr: int, dtype: int, plan_out: Plan, plan_in: Plan, stream: int = 0) -> int:
    """Two-sided processing for callers that cannot allocate device memory (fixed memory
    pools, device budgets owned by another framework): the transposed copy of W lives in a
    32 MiB array inside the library instead of a buffer obtained at call time.  Returns the
    status code (0 = ok, 11 = W larger than the fixed capacity) instead of raising, so a
    caller can fall back to ``harp_apply_two_sided`` with its own scratch."""
    return int(lib().harp_apply_two_sided_static(w_ptr, int(dtype), plan_out.handle, plan_in.handle,
                                                 stream or None))


def harp_two_sided_static_capacity_bytes() -> int:
    return int(lib().harp_two_sided_static_capacity_bytes())


def harp_two_sided_scratch_bytes(plan_out: Plan, plan_in: Plan, dtype: int) -> int:
    return int(lib().harp_two_sided_scratch_bytes(plan_out.handle, plan_in.handle, int(dtype)))


def harp_plan_n_params(plan: Plan) -> int:
    return int(lib().harp_plan_n_params(plan.handle))


def harp_grad_blocks(plan: Plan, x_ptr: int, gy_ptr: int, n_rows: int, dtype: int, grad_ptr: int,
                     accumulate: bool = False, stream: int = 0) -> None:
    """dL/d(block kernels) for y = x Q and G = dL/dy; grad_ptr: DEVICE float[harp_plan_n_params(plan)]."""
    st = lib().harp_grad_blocks(plan.handle, x_ptr, gy_ptr, int(n_rows), int(dtype), grad_ptr,
                                1 if accumulate else 0, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_grad_blocks")


def harp_weight_incoherence(a_ptr: int, m: int, n: int, dtype: int, out_ptr: int, stream: int = 0) -> None:
    """Eq. 4 on a DEVICE m x n matrix; out_ptr: DEVICE double[4] (result in [0])."""
    st = lib().harp_weight_incoherence(a_ptr, int(m), int(n), int(dtype), out_ptr, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_weight_incoherence")


def harp_offblock_energy(h_ptr: int, n: int, block: int, dtype: int, out_ptr: int, stream: int = 0) -> None:
    """Eq. 15 on a DEVICE n x n matrix with contiguous blocks of `block`; out_ptr: DEVICE double[4]."""
    st = lib().harp_offblock_energy(h_ptr, int(n), int(block), int(dtype), out_ptr, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_offblock_energy")


def harp_diag_weighted_error(wt_ptr: int, wq_ptr: int, d_out: int, d_in: int, dtype: int, h_ptr: int, h_dtype: int,
                             out_ptr: int, stream: int = 0) -> None:
    """Eq. 14 for DEVICE Wt, Wq (d_out x d_in) and H (d_in x d_in, diagonal only); out_ptr: DEVICE double[4]."""
    st = lib().harp_diag_weighted_error(wt_ptr, wq_ptr, int(d_out), int(d_in), int(dtype), h_ptr, int(h_dtype),
                                        out_ptr, stream or None)
    if st != HARP_OK:
        raise HarpError(st, "harp_diag_weighted_error")


def harp_apply_host(plan: Plan, host_ptr: int, n_rows: int, dtype: int, transpose: bool = False) -> None:
    """host_ptr: host address (pinned for full speed) of n_rows x d elements, in place."""
    st = lib().harp_apply_host(plan.handle, host_ptr, int(n_rows), int(dtype), 1 if transpose else 0)
    if st != HARP_OK:
        raise HarpError(st, "harp_apply_host")


def shard_rows(n_rows: int, rank: int, world: int):
    """Contiguous row range [start, stop) of `rank` when a batch is split over `world` ranks.
    Rows are independent, so ranks need no collective on the data path."""
    base, rem = divmod(int(n_rows), int(world))
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)


# ---- torch conveniences (device memory and streams only) ----

def _torch_dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return HARP_F32
    if t.dtype == torch.bfloat16:
        return HARP_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def apply_(plan: Plan, x, transpose: bool = False, kernel: int = KERNEL_AUTO):
    """In-place apply to a contiguous CUDA tensor [n_rows, d] on torch's current stream."""
    import torch
    assert x.is_cuda and x.is_contiguous() and x.dim() == 2 and x.shape[1] == plan.d
    harp_apply(plan, x.data_ptr(), x.shape[0], _torch_dtype_code(x), transpose,
               torch.cuda.current_stream().cuda_stream, kernel)
    return x


def two_sided_(w, plan_out: Plan, plan_in: Plan, scratch=None):
    import torch
    assert w.is_cuda and w.is_contiguous() and w.shape == (plan_out.d, plan_in.d)
    harp_apply_two_sided(w.data_ptr(), _torch_dtype_code(w), plan_out, plan_in,
                         0 if scratch is None else scratch.data_ptr(),
                         torch.cuda.current_stream().cuda_stream)
    return w
