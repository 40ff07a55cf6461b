"""The tensor-memory kernels (HARP_KERNEL_TMEM: tcgen05.mma on 128-row tiles, operands in tensor
memory, bulk tensor copies) against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest

import paper_2605_29843_b200 as harp
from oracle import harp_oracle as orc
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import TOL, gpu_apply, host_rows, promote

pytestmark = pytest.mark.gpu


def _check(spec, n_rows, seed, transpose):
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(seed)
    xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
    x64 = promote(xh, "bf16")
    got, guards = gpu_apply(plan, xh, "bf16", transpose=transpose, kernel=harp.KERNEL_TMEM)
    assert harp.harp_plan_error_word(plan) == 0
    assert guards
    want = orc.transpose(oplan, x64) if transpose else orc.forward(oplan, x64)
    assert orc.rel_err_rows(got, want) <= TOL["bf16"]
    return got, want


@pytest.mark.parametrize("transpose", [False, True])
@pytest.mark.parametrize("radices", [(16, 16), (4, 4, 4, 4), (2, 8, 4, 4), (2, 2, 2, 2, 16)])
@pytest.mark.parametrize("n_rows", [128, 1, 300])
def test_two_digits(radices, n_rows, transpose):
    spec = wl.tiny_plan(50, radices, kind="qr", perm="identity", signs=True)
    _check(spec, n_rows, 51, transpose)


@pytest.mark.parametrize("transpose", [False, True])
@pytest.mark.parametrize("perm", ["identity", "digit_reversal"])
@pytest.mark.parametrize("radices", [(4,) * 6, (16, 16, 16), (8, 2, 4, 4, 2, 8)])
def test_three_digits(radices, perm, transpose):
    spec = wl.make_plan(52, 4096, radices, "qr", perm=perm, signs=True)
    _check(spec, 389, 53, transpose)            # three row tiles with a ragged last one


def test_identity_blocks_move_the_bits_exactly():
    """Identity blocks: the apply is the sign flip and the gather, bit for bit (a3 of the path)."""
    for perm in ("identity", "digit_reversal"):
        spec = wl.make_plan(54, 4096, (4,) * 6, "identity", perm=perm, signs=True)
        plan = harp.plan_from_spec(spec)
        rng = np.random.default_rng(55)
        xh = host_rows(rng.standard_normal((200, 4096)), "bf16")
        got, ok = gpu_apply(plan, xh, "bf16", kernel=harp.KERNEL_TMEM)
        assert ok and harp.harp_plan_error_word(plan) == 0
        x64 = promote(xh, "bf16")
        want = (x64 * spec.signs)[:, spec.perm] if spec.perm is not None else x64 * spec.signs
        assert np.array_equal(got, want)
        back, ok = gpu_apply(plan, xh, "bf16", transpose=True, kernel=harp.KERNEL_TMEM)
        inv = np.empty_like(x64)
        if spec.perm is not None:
            inv[:, spec.perm] = x64
        else:
            inv = x64
        assert ok and np.array_equal(back, inv * spec.signs)


def test_a_permutation_that_relabels_inside_the_digits():
    """Any permutation that moves whole 16-ary digits and relabels their values is taken."""
    rng = np.random.default_rng(56)
    t0, t1, t2 = (rng.permutation(16) for _ in range(3))
    i = np.arange(4096)
    perm = (t0[i % 16] + 16 * t1[(i // 16) % 16] + 256 * t2[i // 256]).astype(np.int32)
    spec = wl.make_plan(57, 4096, (4,) * 6, "qr", perm="identity", signs=True)
    spec.perm = perm
    _check(spec, 130, 58, False)
    _check(spec, 130, 58, True)


def test_unsupported_shapes_are_refused():
    spec = wl.tiny_plan(59, (8, 8, 7), perm="random")
    plan = harp.plan_from_spec(spec)
    import torch
    x = torch.zeros((4, spec.d), dtype=torch.bfloat16, device="cuda")
    st = harp.lib().harp_apply_ex(plan.handle, x.data_ptr(), 4, harp.HARP_BF16, 0, harp.KERNEL_TMEM, None)
    assert st == 8


def test_cfg2_full_rows_sampled():
    """cfg2 at 16384 rows in the launch configuration the bench times: sampled rows against the oracle."""
    w = wl.config(2)
    spec, data = w.plans["q"], w.data["x"]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    xh = data.rows(0, data.n_rows)
    rows = np.r_[0:3, 127:130, 8191:8194, data.n_rows - 3:data.n_rows]
    for transpose in (False, True):
        got, ok = gpu_apply(plan, xh, "bf16", transpose=transpose, kernel=harp.KERNEL_TMEM)
        assert ok and harp.harp_plan_error_word(plan) == 0
        x64 = promote(xh[rows], "bf16")
        want = orc.transpose(oplan, x64) if transpose else orc.forward(oplan, x64)
        assert orc.rel_err_rows(got[rows], want) <= TOL["bf16"]


@pytest.mark.parametrize("transpose", [False, True])
@pytest.mark.parametrize("cfg", [3, 4])
def test_wide_rows_take_the_slab_pass(cfg, transpose):
    """cfg3 (2^8 x 43) and cfg4 (16, 16, 8, 7): the stages below stride 256 run in the tensor-memory kernel,
    the rest in the column-group kernels; 1300 rows (ten full 128-row tiles and a ragged one), every
    element against the oracle."""
    w = wl.config(cfg)
    spec, data = w.plans["q"], w.data["x"]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    xh = data.rows(0, 1300)
    before = harp.harp_launch_count()
    got, ok = gpu_apply(plan, xh, "bf16", transpose=transpose)
    assert ok and harp.harp_plan_error_word(plan) == 0
    assert harp.harp_launch_count() - before == 2
    x64 = promote(xh, "bf16")
    want = orc.transpose(oplan, x64) if transpose else orc.forward(oplan, x64)
    assert orc.rel_err_rows(got, want) <= TOL["bf16"]
