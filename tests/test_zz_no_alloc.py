"""The allocation-free two-sided entry point, for callers that cannot allocate device
memory when they call (fixed pools, budgets owned by another framework).  It must give
what harp_apply_two_sided gives, on repeated calls that reuse the library's fixed scratch
array, and must refuse matrices larger than that array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2605_29843_b200 as harp
from oracle import harp_oracle as orc
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import TOL, promote, to_device, to_host_f64

pytestmark = pytest.mark.gpu


def _case(seed, out_radices, in_radices, dtype):
    p_out = wl.tiny_plan(seed, out_radices, perm="random")
    p_in = wl.tiny_plan(seed + 1, in_radices, perm="random")
    rng = np.random.default_rng(seed)
    w32 = rng.standard_normal((p_out.d, p_in.d)).astype(np.float32)
    wh = w32 if dtype == "f32" else wl.f32_to_bf16_bits(w32)
    return harp.plan_from_spec(p_out), harp.plan_from_spec(p_in), wh


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_matches_the_allocating_entry_point_twice_in_a_row(dtype):
    code = harp.HARP_F32 if dtype == "f32" else harp.HARP_BF16
    stream = torch.cuda.current_stream().cuda_stream
    # two different shapes back to back: the second call finds the first call's leftovers
    for seed, out_r, in_r in ((3, (8, 8, 2), (8, 8, 7)), (5, (4, 4, 4, 3), (16, 16, 2))):
        plan_out, plan_in, wh = _case(seed, out_r, in_r, dtype)
        ref = to_device(wh, dtype)
        harp.two_sided_(ref, plan_out, plan_in)                    # existing entry point
        got = to_device(wh, dtype)
        st = harp.harp_apply_two_sided_static(got.data_ptr(), code, plan_out, plan_in, stream)
        assert st == harp.HARP_OK
        torch.cuda.synchronize()
        a, b = to_host_f64(got), to_host_f64(ref)
        scale = np.linalg.norm(b, axis=1).min()
        assert np.max(np.abs(a - b)) / scale <= TOL[dtype]
        # and once more on the result of the first call (second call in a row)
        st = harp.harp_apply_two_sided_static(got.data_ptr(), code, plan_out, plan_in, stream)
        assert st == harp.HARP_OK
        harp.two_sided_(ref, plan_out, plan_in)
        torch.cuda.synchronize()
        a, b = to_host_f64(got), to_host_f64(ref)
        assert np.max(np.abs(a - b)) / np.linalg.norm(b, axis=1).min() <= TOL[dtype]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("perm", ["random", "identity"])
def test_static_scratch_against_the_oracle(dtype, perm):
    """The fixed-scratch entry point against the fp64 definition Q_out^T W Q_in itself (not against the
    other entry point, which could share a mistake with it), with permuted and with identity plans:
    identity plans are the ones the allocating entry point sends down its column kernels, so here the
    two take different routes.  Called twice on fresh copies, so the second call runs on leftovers."""
    code = harp.HARP_F32 if dtype == "f32" else harp.HARP_BF16
    stream = torch.cuda.current_stream().cuda_stream
    p_out = wl.tiny_plan(11, (8, 8, 2), perm=perm)
    p_in = wl.tiny_plan(12, (16, 16, 7), perm=perm)
    plan_out, plan_in = harp.plan_from_spec(p_out), harp.plan_from_spec(p_in)
    rng = np.random.default_rng(13)
    w32 = rng.standard_normal((p_out.d, p_in.d)).astype(np.float32)
    wh = w32 if dtype == "f32" else wl.f32_to_bf16_bits(w32)
    want = orc.two_sided(orc.OraclePlan.from_spec(p_out), orc.OraclePlan.from_spec(p_in), promote(wh, dtype))
    scale = np.linalg.norm(want, axis=1).min()
    for _ in range(2):
        got = to_device(wh, dtype)
        assert harp.harp_apply_two_sided_static(got.data_ptr(), code, plan_out, plan_in, stream) == harp.HARP_OK
        torch.cuda.synchronize()
        # two sides, each within the one-sided tolerance
        assert np.max(np.abs(to_host_f64(got) - want)) / scale <= 2 * TOL[dtype]


def test_static_scratch_takes_a_matrix_of_exactly_the_capacity_and_allocates_nothing():
    """W of exactly 32 MiB (4096 x 4096 bf16) is accepted; after a first call has loaded the module and
    looked the array's address up, a further call leaves the device's free memory and torch's
    allocator counters where they were."""
    d = 4096
    spec = wl.make_plan(14, d, (8, 8, 8, 8), "qr", signs=True)
    plan = harp.plan_from_spec(spec)
    assert d * d * 2 == harp.harp_two_sided_static_capacity_bytes()
    w = torch.randn((d, d), device="cuda").to(torch.bfloat16)
    stream = torch.cuda.current_stream().cuda_stream
    assert harp.harp_apply_two_sided_static(w.data_ptr(), harp.HARP_BF16, plan, plan, stream) == harp.HARP_OK
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    stats0 = torch.cuda.memory_stats()["allocation.all.allocated"]
    assert harp.harp_apply_two_sided_static(w.data_ptr(), harp.HARP_BF16, plan, plan, stream) == harp.HARP_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == stats0
    # the map is orthogonal on both sides: the Frobenius norm survives two applications
    assert np.isfinite(float(w.float().norm()))


def test_static_scratch_rejects_what_does_not_fit():
    cap = harp.harp_two_sided_static_capacity_bytes()
    assert cap == 32 << 20
    d = 8192                                   # 8192 x 8192 bf16 = 128 MiB > capacity
    spec = wl.make_plan(0, d, (8, 8, 8, 8, 2), "identity", signs=False)
    plan = harp.plan_from_spec(spec)
    w = torch.zeros((16, 16), dtype=torch.bfloat16, device="cuda")     # never touched
    before = harp.harp_launch_count()
    st = harp.harp_apply_two_sided_static(w.data_ptr(), harp.HARP_BF16, plan, plan, 0)
    assert st == 11 and harp.status_string(st) == "exceeds a fixed capacity"
    assert harp.harp_launch_count() == before
