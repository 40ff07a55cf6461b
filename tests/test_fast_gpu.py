"""Tensor-core path (explicit HARP_KERNEL_FAST) against the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2605_29843_b200 as harp
from oracle import harp_oracle as orc
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import TOL, gpu_apply, host_rows, promote

pytestmark = pytest.mark.gpu

SUPPORTED = [
    ((4, 4), "identity"), ((4, 4, 4, 4), "identity"), ((4,) * 6, "identity"), ((4,) * 6, "digit_reversal"),
    ((2,) * 11, "identity"), ((2,) * 11, "digit_reversal"), ((8, 8), "identity"), ((8, 8, 8, 8), "identity"),
    ((16, 16, 8), "identity"), ((16, 16, 8), "digit_reversal"), ((2, 8, 4, 4, 8), "identity"),
    ((4, 4, 2, 2, 2, 2, 16), "digit_reversal"), ((16, 16, 16), "digit_reversal"),
]


@pytest.mark.parametrize("radices,perm", SUPPORTED)
@pytest.mark.parametrize("kind", ["qr", "identity"])
def test_fast_kernel_matches_oracle(radices, perm, kind):
    spec = wl.make_plan(23, int(np.prod(radices)), radices, kind, perm=perm, signs=True)
    oplan = orc.OraclePlan.from_spec(spec)
    plan = harp.plan_from_spec(spec)
    rng = np.random.default_rng(8)
    for n_rows in (1, 16, 37, 600):
        xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
        x64 = promote(xh, "bf16")
        for tr in (False, True):
            got, guards = gpu_apply(plan, xh, "bf16", tr, harp.KERNEL_FAST)
            want = orc.transpose(oplan, x64) if tr else orc.forward(oplan, x64)
            assert guards
            if kind == "identity":
                assert np.array_equal(got, want)            # sign + gather must be bit exact
            else:
                assert orc.rel_err_rows(got, want) <= TOL["bf16"]


@pytest.mark.parametrize("radices,perm", [((4,) * 6, "digit_reversal"), ((4,) * 6, "identity"), ((16, 16, 8), "digit_reversal")])
def test_several_tiles_per_cta_and_a_ragged_last_tile(radices, perm):
    """More tiles than SMs, so that a CTA works through several tiles, and row counts that leave the last tile
    partly empty.  For the largest count a sample of rows (both ends of the batch and rows in between) is
    compared, otherwise every row."""
    spec = wl.make_plan(29, int(np.prod(radices)), radices, "qr", perm=perm, signs=True)
    oplan = orc.OraclePlan.from_spec(spec)
    plan = harp.plan_from_spec(spec)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rng = np.random.default_rng(12)
    for n_rows in (16 * sms * 2 + 7, 16 * sms + 16 * 3 + 1, 12 * sms * 6 + 12 * 5 + 5):
        xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
        pick = np.arange(n_rows)
        if n_rows > 6000:
            pick = np.unique(np.concatenate([np.arange(40), np.arange(n_rows - 40, n_rows), rng.integers(0, n_rows, 300)]))
        x64 = promote(xh[pick], "bf16")
        for tr in (False, True):
            got, guards = gpu_apply(plan, xh, "bf16", tr, harp.KERNEL_FAST)
            want = orc.transpose(oplan, x64) if tr else orc.forward(oplan, x64)
            assert guards
            assert orc.rel_err_rows(got[pick], want) <= TOL["bf16"]


@pytest.mark.parametrize("radices,perm,dtype", [((16, 16, 8, 7), "identity", "bf16"), ((4,) * 6, "random", "bf16"),
                                                ((4,) * 6, "identity", "f32"), ((2,) * 9, "identity", "bf16")])
def test_fast_kernel_reports_unsupported(radices, perm, dtype):
    spec = wl.make_plan(3, int(np.prod(radices)), radices, "qr", perm=perm)
    plan = harp.plan_from_spec(spec)
    x = torch.zeros((16, spec.d), device="cuda", dtype=torch.float32 if dtype == "f32" else torch.bfloat16)
    st = harp.lib().harp_apply_ex(plan.handle, x.data_ptr(), 16, 0 if dtype == "f32" else 1, 0, harp.KERNEL_FAST, None)
    assert st == harp.HARP_ERR_UNSUPPORTED
    harp.apply_(plan, x)                                    # AUTO still works (generic kernel)
    torch.cuda.synchronize()


SPLIT = [(4, 4, 4, 4), (8, 8, 8, 8), (16, 16, 8), (2,) * 11, (16, 16, 8, 7), (8, 8, 8, 8, 7), (8, 8, 8, 8, 2),
         (16, 4, 3, 5), (8, 2, 2, 2, 3), (16, 16, 2, 2, 5), (2,) * 8 + (43,), (16, 16, 17), (8, 8, 8, 33),
         (4, 4, 4, 4, 64), (8, 8, 21, 3)]


@pytest.mark.parametrize("radices", SPLIT)
@pytest.mark.parametrize("kind", ["qr", "identity"])
def test_split_kernel_matches_oracle(radices, kind):
    spec = wl.make_plan(29, int(np.prod(radices)), radices, kind, perm="identity", signs=True)
    oplan = orc.OraclePlan.from_spec(spec)
    plan = harp.plan_from_spec(spec)
    rng = np.random.default_rng(9)
    big = 2100 if spec.d > 10000 else 600            # more rows than one L2 chunk for the wide plans
    for n_rows in (1, 16, 17, 33, 37, big):          # 17 and 33: just past the 16- and 32-row tiles a small batch takes
        xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
        x64 = promote(xh, "bf16")
        for tr in (False, True):
            got, guards = gpu_apply(plan, xh, "bf16", tr, harp.KERNEL_SPLIT)
            want = orc.transpose(oplan, x64) if tr else orc.forward(oplan, x64)
            assert guards
            if kind == "identity":
                assert np.array_equal(got, want)
            else:
                assert orc.rel_err_rows(got, want) <= TOL["bf16"]


@pytest.mark.parametrize("radices", [(16, 16, 8, 7), (8, 8, 8, 8, 7), (8, 8, 8, 8)])
def test_split_kernel_with_dense_upper_block(radices, monkeypatch):
    monkeypatch.setenv("HARP_UPPER_DENSE", "1")
    spec = wl.make_plan(31, int(np.prod(radices)), radices, "qr", perm="identity", signs=True)
    oplan = orc.OraclePlan.from_spec(spec)
    plan = harp.plan_from_spec(spec)
    rng = np.random.default_rng(10)
    for n_rows in (5, 100):
        xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
        x64 = promote(xh, "bf16")
        for tr in (False, True):
            got, guards = gpu_apply(plan, xh, "bf16", tr, harp.KERNEL_SPLIT)
            want = orc.transpose(oplan, x64) if tr else orc.forward(oplan, x64)
            assert guards and orc.rel_err_rows(got, want) <= TOL["bf16"]


SPLIT_PERM = [((4,) * 6, "digit_reversal"), ((16, 16, 8, 7), "random"), ((8, 8, 8, 8, 7), "random"), ((2,) * 8 + (43,), "random"),
              ((16, 16, 8, 7), "digit_reversal"), ((8, 8, 8, 5), "random")]


@pytest.mark.parametrize("radices,perm", SPLIT_PERM)
@pytest.mark.parametrize("kind", ["qr", "identity"])
def test_split_kernel_with_a_permutation(radices, perm, kind):
    """Plans with a permutation: the two passes plus the row-gather kernel (three launches, or two when
    one pass covers all stages), every element against the oracle; identity blocks leave the sign flip
    and the gather, which must be exact."""
    spec = wl.make_plan(33, int(np.prod(radices)), radices, kind, perm=perm, signs=True)
    oplan = orc.OraclePlan.from_spec(spec)
    plan = harp.plan_from_spec(spec)
    rng = np.random.default_rng(11)
    for n_rows in (1, 37, 1300):
        xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
        x64 = promote(xh, "bf16")
        for tr in (False, True):
            before = harp.harp_launch_count()
            got, guards = gpu_apply(plan, xh, "bf16", tr, harp.KERNEL_SPLIT)
            assert harp.harp_launch_count() - before <= 3
            assert harp.harp_plan_error_word(plan) == 0
            want = orc.transpose(oplan, x64) if tr else orc.forward(oplan, x64)
            assert guards
            if kind == "identity":
                assert np.array_equal(got, want)
            else:
                assert orc.rel_err_rows(got, want) <= TOL["bf16"]


def test_auto_takes_the_tensor_core_route_for_permuted_wide_rows():
    """cfg4's schedule with a random permutation: AUTO = gather + two tensor-core passes, not the
    per-coordinate kernel (which takes one launch)."""
    spec = wl.make_plan(35, 14336, (16, 16, 8, 7), "qr", perm="random", signs=True)
    oplan = orc.OraclePlan.from_spec(spec)
    plan = harp.plan_from_spec(spec)
    rng = np.random.default_rng(12)
    xh = host_rows(rng.standard_normal((1100, spec.d)), "bf16")
    x64 = promote(xh, "bf16")
    for tr in (False, True):
        before = harp.harp_launch_count()
        got, guards = gpu_apply(plan, xh, "bf16", tr)
        assert harp.harp_launch_count() - before == 3
        want = orc.transpose(oplan, x64) if tr else orc.forward(oplan, x64)
        assert guards and orc.rel_err_rows(got, want) <= TOL["bf16"]


@pytest.mark.parametrize("radices,perm", [((2,) * 8 + (67,), "identity"), ((7, 2, 4), "identity"), ((7, 2, 4), "random")])
def test_split_kernel_reports_unsupported(radices, perm):
    spec = wl.make_plan(3, int(np.prod(radices)), radices, "qr", perm=perm)
    plan = harp.plan_from_spec(spec)
    x = torch.zeros((16, spec.d), device="cuda", dtype=torch.bfloat16)
    st = harp.lib().harp_apply_ex(plan.handle, x.data_ptr(), 16, 1, 0, harp.KERNEL_SPLIT, None)
    assert st == harp.HARP_ERR_UNSUPPORTED


@pytest.mark.parametrize("out_radices,in_radices", [((8, 8, 8, 8, 2), (4, 4, 4)), ((16, 16, 8, 7), (8, 9)),
                                                    ((8, 8, 8, 8, 7), (8, 8)), ((4, 4, 4), (16, 16, 8)),
                                                    ((16, 4, 3, 5), (8, 5)), ((8, 8, 8, 8), (8, 8, 8, 8))])
def test_two_sided_with_column_kernels(out_radices, in_radices):
    """plan_out without permutation and d_in a multiple of 8: the column side runs in place."""
    from oracle import c_oracle
    from harp_testlib import to_device, to_host_f64
    p_out = wl.make_plan(51, int(np.prod(out_radices)), out_radices, "qr", perm="identity", signs=True)
    p_in = wl.make_plan(52, int(np.prod(in_radices)), in_radices, "qr", perm="identity", signs=True)
    rng = np.random.default_rng(12)
    wh = host_rows(rng.standard_normal((p_out.d, p_in.d)), "bf16")
    w64 = promote(wh, "bf16")
    wd = to_device(wh, "bf16")
    before = harp.harp_launch_count()
    harp.two_sided_(wd, harp.plan_from_spec(p_out), harp.plan_from_spec(p_in))
    torch.cuda.synchronize()
    assert harp.harp_launch_count() - before <= 4          # no transposes: at most two passes per side
    want = c_oracle.two_sided(c_oracle.CPlan(p_out), c_oracle.CPlan(p_in), w64)
    got = to_host_f64(wd)
    scale = np.minimum(np.linalg.norm(want, axis=1, keepdims=True), np.linalg.norm(want, axis=0, keepdims=True))
    assert np.max(np.abs(got - want) / scale) <= 2 * TOL["bf16"]
