"""Diagnostics kernels (Eq. 4, Eq. 14, Eq. 15) on the GPU against the numpy oracle.
The kernels accumulate in fp64 over the same rounded inputs the oracle reads, so the results
agree to the rounding of the summation order: relative 1e-11."""
import numpy as np
import pytest
import torch

import paper_2605_29843_b200 as harp
from oracle import harp_diagnostics as od
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import host_rows, promote, to_device

pytestmark = pytest.mark.gpu

REL = 1e-11
DT = {"f32": harp.HARP_F32, "bf16": harp.HARP_BF16}


def _out():
    return torch.full((4,), 7.0, dtype=torch.float64, device="cuda")     # the call must zero it itself


def _matrix(rng, m, n, dtype, heavy=False):
    a = rng.standard_t(3, size=(m, n)) if heavy else rng.standard_normal((m, n))
    h = host_rows(a, dtype)
    return h, promote(h, dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m,n", [(1, 8), (5, 17), (64, 256), (300, 1000), (129, 2048 + 8)])
def test_weight_incoherence(dtype, m, n):
    rng = np.random.default_rng(m * 1000 + n)
    h, a64 = _matrix(rng, m, n, dtype, heavy=True)
    out = _out()
    a_d = to_device(h, dtype)
    harp.harp_weight_incoherence(a_d.data_ptr(), m, n, DT[dtype], out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    got = out.cpu().numpy()
    assert got[0] == pytest.approx(od.weight_incoherence(a64), rel=REL)
    assert got[1] == np.max(np.abs(a64))                                  # a maximum is exact
    assert got[2] == pytest.approx(np.sum(a64 * a64), rel=REL)


def test_weight_incoherence_unaligned_view_and_zero_matrix():
    rng = np.random.default_rng(9)
    h, a64 = _matrix(rng, 33, 24, "f32")
    buf = torch.zeros(33 * 24 + 1, dtype=torch.float32, device="cuda")
    buf[1:] = torch.from_numpy(h).cuda().flatten()                        # 4-byte aligned only
    out = _out()
    harp.harp_weight_incoherence(buf[1:].data_ptr(), 33, 24, harp.HARP_F32, out.data_ptr())
    assert out.cpu().numpy()[0] == pytest.approx(od.weight_incoherence(a64), rel=REL)
    z = torch.zeros((16, 16), dtype=torch.bfloat16, device="cuda")
    harp.harp_weight_incoherence(z.data_ptr(), 16, 16, harp.HARP_BF16, out.data_ptr())
    assert out.cpu().numpy()[0] == 0.0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,block", [(8, 8), (8, 1), (10, 4), (96, 8), (512, 16), (1000, 24), (2048, 8)])
def test_offblock_energy(dtype, n, block):
    rng = np.random.default_rng(n + block)
    x = rng.standard_normal((max(4, n // 8), n))
    h, h64 = host_rows(x.T @ x / x.shape[0], dtype), None
    h64 = promote(h, dtype)
    out = _out()
    h_d = to_device(h, dtype)
    harp.harp_offblock_energy(h_d.data_ptr(), n, block, DT[dtype], out.data_ptr())
    got = out.cpu().numpy()
    want = od.offblock_energy(h64, block)
    if want == 0.0:
        assert abs(got[0]) <= 1e-12 * np.sum(h64 * h64) / n ** 2
    else:
        assert got[0] == pytest.approx(want, rel=1e-9)                    # a difference of two sums
    assert got[2] == pytest.approx(np.sum(h64 * h64), rel=REL)


@pytest.mark.parametrize("dtype,h_dtype", [("bf16", "f32"), ("f32", "f32"), ("bf16", "bf16")])
@pytest.mark.parametrize("d_out,d_in", [(3, 8), (17, 40), (256, 1024), (100, 1000 + 4)])
def test_diag_weighted_error(dtype, h_dtype, d_out, d_in):
    rng = np.random.default_rng(d_out + d_in)
    wt_h, wt64 = _matrix(rng, d_out, d_in, dtype)
    wq_h = host_rows(np.round(wt64 * 4) / 4, dtype)                       # a stand-in quantizer: a grid of step 1/4
    wq64 = promote(wq_h, dtype)
    x = rng.standard_normal((32, d_in)) * (1.0 + 5.0 * (rng.random(d_in) < 0.02))
    hh = host_rows(x.T @ x / 32.0, h_dtype)
    out = _out()
    wt_d, wq_d, h_d = to_device(wt_h, dtype), to_device(wq_h, dtype), to_device(hh, h_dtype)
    harp.harp_diag_weighted_error(wt_d.data_ptr(), wq_d.data_ptr(), d_out, d_in, DT[dtype], h_d.data_ptr(), DT[h_dtype],
                                  out.data_ptr())
    got = out.cpu().numpy()
    assert got[0] == pytest.approx(od.diag_weighted_error(wt64, wq64, promote(hh, h_dtype)), rel=REL)


def test_diagnostics_reject_bad_arguments():
    out = _out()
    a = torch.zeros((4, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(harp.HarpError):
        harp.harp_weight_incoherence(0, 4, 4, harp.HARP_F32, out.data_ptr())
    with pytest.raises(harp.HarpError):
        harp.harp_weight_incoherence(a.data_ptr(), 0, 4, harp.HARP_F32, out.data_ptr())
    with pytest.raises(harp.HarpError):
        harp.harp_offblock_energy(a.data_ptr(), 4, 5, harp.HARP_F32, out.data_ptr())
    with pytest.raises(harp.HarpError):
        harp.harp_offblock_energy(a.data_ptr(), 4, 2, 7, out.data_ptr())


def test_incoherence_of_a_processed_weight_full_size():
    """cfg5-sized use: mu_W of W before and after two-sided processing with the cfg5 plans; the
    Frobenius norm is preserved by the orthogonal maps, and the kernel agrees with numpy on W~."""
    w5 = wl.config(5)
    plan_out, plan_in = harp.plan_from_spec(w5.plans["out"]), harp.plan_from_spec(w5.plans["in"])
    d_out, d_in = w5.plans["out"].d, w5.plans["in"].d
    g = torch.Generator(device="cuda").manual_seed(5)
    W = (torch.randn((d_out, d_in), device="cuda", generator=g) * 0.02)
    W[:, ::997] *= 30.0                                                   # outlier channels
    W = W.to(torch.bfloat16)
    out0, out1 = _out(), _out()
    harp.harp_weight_incoherence(W.data_ptr(), d_out, d_in, harp.HARP_BF16, out0.data_ptr())
    harp.two_sided_(W, plan_out, plan_in)
    harp.harp_weight_incoherence(W.data_ptr(), d_out, d_in, harp.HARP_BF16, out1.data_ptr())
    torch.cuda.synchronize()
    before, after = out0.cpu().numpy(), out1.cpu().numpy()
    assert after[2] == pytest.approx(before[2], rel=2e-2)                 # ||W||_F^2 up to bf16 rounding of W~
    assert after[0] < before[0]                                           # the outliers are spread out
    w64 = W.double()
    mu = float(np.sqrt(d_out * d_in) * w64.abs().max().item() / w64.pow(2).sum().sqrt().item())
    assert after[0] == pytest.approx(mu, rel=1e-9)
