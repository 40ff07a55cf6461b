"""Block kernels rebuilt from stored parameters on the GPU (harp_blocks_from_theta_device) against
the plan-side oracle: Givens rotation and Cayley map times the mixer, from fp32 parameters and from
int8 parameters with one scale per block."""
import numpy as np
import pytest
import torch

import paper_2605_29843_b200 as harp
from oracle import harp_params as prm
from paper_2605_29843_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _mixer(b, rng):
    if b & (b - 1) == 0:
        return None
    return wl.qr_orthogonal(rng, 1, b)[0].astype(np.float32)


@pytest.mark.parametrize("int8", [False, True])
@pytest.mark.parametrize("b", [2, 3, 4, 5, 7, 8, 16, 43])
def test_device_blocks_match_the_oracle(b, int8):
    rng = np.random.default_rng(100 + b)
    n = 37
    npar = prm.n_params(b)
    theta = rng.normal(0.0, 0.4 if b > 2 else 2.0, (n, npar)).astype(np.float32)
    mixer = _mixer(b, rng)
    out = torch.full((n, b, b), 9.0, dtype=torch.float32, device="cuda")
    mx = None if mixer is None else torch.from_numpy(mixer).cuda()
    if int8:
        q, s = prm.quantize_theta(theta)
        s32 = s.astype(np.float32)
        want = prm.blocks_from_theta(b, prm.dequantize_theta(q, s32), None if mixer is None else mixer.astype(np.float64))
        tq, sc = torch.from_numpy(q).cuda(), torch.from_numpy(s32).cuda()
        harp.harp_blocks_from_theta_device(b, n, 0, tq.data_ptr(), sc.data_ptr(), 0 if mx is None else mx.data_ptr(),
                                           out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    else:
        want = prm.blocks_from_theta(b, theta, None if mixer is None else mixer.astype(np.float64))
        th = torch.from_numpy(theta).cuda()
        harp.harp_blocks_from_theta_device(b, n, th.data_ptr(), 0, 0, 0 if mx is None else mx.data_ptr(),
                                           out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got - want)) <= 2e-7
    # orthogonal to fp32 rounding
    assert np.max(np.abs(got @ np.swapaxes(got, 1, 2) - np.eye(b))) <= 1e-5


def test_device_and_host_reconstruction_agree_and_limits():
    b, n = 16, 50
    rng = np.random.default_rng(7)
    theta = rng.normal(0.0, 0.3, (n, prm.n_params(b))).astype(np.float32)
    host = np.empty((n, b, b), dtype=np.float32)
    st = harp.lib().harp_blocks_from_theta(b, n, theta.ctypes.data, None, None, None, host.ctypes.data)
    assert st == harp.HARP_OK
    out = torch.empty((n, b, b), dtype=torch.float32, device="cuda")
    th = torch.from_numpy(theta).cuda()
    harp.harp_blocks_from_theta_device(b, n, th.data_ptr(), 0, 0, 0, out.data_ptr())
    torch.cuda.synchronize()
    assert np.max(np.abs(out.cpu().numpy() - host)) <= 1.2e-7      # both round an fp64 result once
    # beyond the device limit, and a radix without a default mixer
    L = harp.lib()
    assert L.harp_theta_device_max_radix() == 54
    assert L.harp_blocks_from_theta_device(55, 1, th.data_ptr(), None, None, None, out.data_ptr(), None) == 8
    assert L.harp_blocks_from_theta_device(3, 1, th.data_ptr(), None, None, None, out.data_ptr(), None) == 1
    assert L.harp_blocks_from_theta_device(4, 0, th.data_ptr(), None, None, None, out.data_ptr(), None) == harp.HARP_OK
