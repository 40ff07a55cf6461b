"""harp_grad_blocks on the GPU against the oracle's chain rule, and against invariants at a
configuration's full dimension."""
import numpy as np
import pytest
import torch

import paper_2605_29843_b200 as harp
from oracle import harp_oracle as orc
from oracle import harp_params as prm
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import host_rows, promote, to_device

pytestmark = pytest.mark.gpu

DT = {"f32": harp.HARP_F32, "bf16": harp.HARP_BF16}


def _gpu_grad(plan, xh, gh, dtype, accumulate=False, init=None):
    n = xh.shape[0]
    x_d, g_d = to_device(xh, dtype), to_device(gh, dtype)
    n_par = harp.harp_plan_n_params(plan)
    out = torch.full((n_par,), 3.0, dtype=torch.float32, device="cuda") if init is None else init.clone()
    harp.harp_grad_blocks(plan, x_d.data_ptr(), g_d.data_ptr(), n, DT[dtype], out.data_ptr(), accumulate,
                          torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64), x_d, g_d


def _flat(grads):
    return np.concatenate([g.ravel() for g in grads])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("radices,perm", [((4,), "identity"), ((2, 2, 2), "random"), ((4, 3, 5), "random"),
                                          ((16, 8, 2), "identity"), ((7, 2), "random"), ((43, 2), "identity")])
def test_grad_blocks_matches_the_oracle(dtype, radices, perm):
    spec = wl.tiny_plan(31, radices, kind="qr", perm=perm, signs=True)
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(32)
    xh = host_rows(rng.standard_normal((29, spec.d)), dtype)
    gh = host_rows(rng.standard_normal((29, spec.d)), dtype)
    got, x_d, g_d = _gpu_grad(plan, xh, gh, dtype)
    want = _flat(orc.grad_blocks(oplan, promote(xh, dtype), promote(gh, dtype)))
    assert got.shape == want.shape == (harp.harp_plan_n_params(plan),)
    # fp32 stage states, fp64 row sums: error relative to the size of the largest entry
    assert np.max(np.abs(got - want)) <= 2e-5 * np.max(np.abs(want))
    # the inputs are not modified
    assert np.array_equal(x_d.cpu().view(torch.int16 if dtype == "bf16" else torch.int32).numpy(),
                          to_device(xh, dtype).cpu().view(torch.int16 if dtype == "bf16" else torch.int32).numpy())


@pytest.mark.parametrize("radices", [(8, 4, 2), (2, 8), (4, 4, 4), (6, 7), (5, 3, 7), (2, 16), (4, 16, 2), (16, 16)])
def test_rows_spanning_several_slices(radices):
    """More rows than one thread block of the block-owner kernels walks, with a ragged last slice
    and a ragged last batch; radix 8 both at stride one and strided."""
    spec = wl.tiny_plan(35, radices, kind="qr", perm="random", signs=True)
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(36)
    xh = host_rows(rng.standard_normal((71, spec.d)), "f32")
    gh = host_rows(rng.standard_normal((71, spec.d)), "f32")
    got, _, _ = _gpu_grad(plan, xh, gh, "f32")
    want = _flat(orc.grad_blocks(oplan, promote(xh, "f32"), promote(gh, "f32")))
    assert np.max(np.abs(got - want)) <= 2e-5 * np.max(np.abs(want))
    again, _, _ = _gpu_grad(plan, xh, gh, "f32")
    assert np.array_equal(got, again)                       # fixed summation order


def test_accumulate_and_row_chunks_add_up():
    spec = wl.tiny_plan(33, (4, 4, 2), kind="qr", perm="random", signs=True)
    plan = harp.plan_from_spec(spec)
    rng = np.random.default_rng(34)
    xh, gh = host_rows(rng.standard_normal((40, 32)), "f32"), host_rows(rng.standard_normal((40, 32)), "f32")
    full, _, _ = _gpu_grad(plan, xh, gh, "f32")
    first, _, _ = _gpu_grad(plan, xh[:15], gh[:15], "f32")
    both, _, _ = _gpu_grad(plan, xh[15:], gh[15:], "f32", accumulate=True,
                           init=torch.from_numpy(first.astype(np.float32)).cuda())
    assert np.max(np.abs(both - full)) <= 1e-5 * np.max(np.abs(full))
    # no rows: the result is zero (or untouched when accumulating)
    n_par = harp.harp_plan_n_params(plan)
    out = torch.full((n_par,), 3.0, dtype=torch.float32, device="cuda")
    harp.harp_grad_blocks(plan, 0, 0, 0, harp.HARP_F32, out.data_ptr())
    assert float(out.abs().max()) == 0.0


def _rows(seed, n, d, dtype):
    rng = np.random.default_rng(seed)
    return host_rows(rng.standard_normal((n, d)), dtype), host_rows(rng.standard_normal((n, d)), dtype)


def test_every_entry_at_full_dimension_cfg2():
    """cfg2's plan (d = 4096, six radix-4 stages, digit-reversal permutation) on 4100 bf16 rows --
    more than one internal row chunk, ragged against every slice size: every entry of every
    stage's gradient against the oracle's chain rule through Algorithm 1."""
    spec = wl.config(2).plans["q"]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    xh, gh = _rows(90, 4100, spec.d, "bf16")
    got, _, _ = _gpu_grad(plan, xh, gh, "bf16")
    want = _flat(orc.grad_blocks(oplan, promote(xh, "bf16"), promote(gh, "bf16")))
    assert got.shape == want.shape
    off = 0
    for t, b in enumerate(spec.radices):                     # per stage, so a quiet stage cannot hide
        n = spec.d * b
        g, w = got[off:off + n], want[off:off + n]
        off += n
        assert np.max(np.abs(g - w)) <= 2e-5 * np.max(np.abs(w)), t


def test_every_entry_at_full_dimension_cfg4():
    """cfg4's plan (d = 14336, radices 16, 16, 8, 7): all entries on 256 rows, and again on a batch
    long enough to cross the internal row chunk."""
    spec = list(wl.config(4).plans.values())[0]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    for seed, n in ((91, 256), (92, 1203)):
        xh, gh = _rows(seed, n, spec.d, "bf16")
        got, _, _ = _gpu_grad(plan, xh, gh, "bf16")
        want = _flat(orc.grad_blocks(oplan, promote(xh, "bf16"), promote(gh, "bf16")))
        off = 0
        for t, b in enumerate(spec.radices):
            m = spec.d * b
            g, w = got[off:off + m], want[off:off + m]
            off += m
            assert np.max(np.abs(g - w)) <= 2e-5 * np.max(np.abs(w)), (n, t)


def test_euler_identity_at_full_dimension():
    """cfg2's plan (d = 4096, six radix-4 stages, digit-reversal permutation): y is homogeneous of
    degree one in the kernels of every stage, so <K_t, dL/dK_t> = sum(y * G) for each t; y comes
    from harp_apply itself."""
    w = wl.config(2)
    spec = w.plans["q"]
    plan = harp.plan_from_spec(spec)
    n = 512
    g = torch.Generator(device="cuda").manual_seed(7)
    x = torch.randn((n, spec.d), device="cuda", generator=g)
    G = torch.randn((n, spec.d), device="cuda", generator=g)
    grad = torch.zeros(harp.harp_plan_n_params(plan), dtype=torch.float32, device="cuda")
    harp.harp_grad_blocks(plan, x.data_ptr(), G.data_ptr(), n, harp.HARP_F32, grad.data_ptr())
    y = x.clone()
    harp.apply_(plan, y)
    L = float((y.double() * G.double()).sum())
    off = 0
    for t, b in enumerate(spec.radices):
        k = torch.from_numpy(np.ascontiguousarray(spec.blocks[t], dtype=np.float32)).cuda().flatten()
        got = float((k.double() * grad[off:off + k.numel()].double()).sum())
        off += k.numel()
        assert got == pytest.approx(L, rel=2e-4), t
    assert off == grad.numel()


@pytest.mark.parametrize("cfg", [3, 4, 5])
def test_euler_identity_on_the_wide_plans(cfg):
    """The wide configurations' plans at full dimension (radices 2 and 43; 16, 16, 8, 7; 8, 8, 8, 8, 2),
    bf16 rows: <K_t, dL/dK_t> = L = sum(y * G) for every stage, with y from the fp64 oracle."""
    w = wl.config(cfg)
    spec = list(w.plans.values())[0]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(80 + cfg)
    n = 96
    xh = host_rows(rng.standard_normal((n, spec.d)), "bf16")
    gh = host_rows(rng.standard_normal((n, spec.d)), "bf16")
    grad, _, _ = _gpu_grad(plan, xh, gh, "bf16")
    L = float(np.sum(orc.forward(oplan, promote(xh, "bf16")) * promote(gh, "bf16")))
    scale = float(np.sqrt(n * spec.d))                      # size of L for independent unit-variance terms
    off = 0
    for t, b in enumerate(spec.radices):
        k = np.asarray(spec.blocks[t], dtype=np.float32).astype(np.float64).ravel()
        got = float(np.dot(k, grad[off:off + k.size]))
        off += k.size
        assert abs(got - L) <= 2e-4 * max(abs(L), scale), (t, b, got, L)
    assert off == grad.size


def test_parameter_gradient_of_a_plan_built_from_theta():
    """One parameter step's worth of Algorithm 3 without the quantizer: plan from theta, L = sum(y * G)
    with y from harp_apply, dL/dK on the GPU, dL/dtheta on the host; compared with central
    differences of the fp64 oracle (theta -> blocks -> forward) on sampled parameters."""
    radices, d = (4, 2, 8), 64
    rng = np.random.default_rng(70)
    theta = [rng.normal(0, 0.3, (d // b, prm.n_params(b))).astype(np.float32) for b in radices]
    perm = rng.permutation(d).astype(np.int32)
    signs = rng.choice(np.array([-1, 1], dtype=np.int8), d)
    plan = harp.harp_plan_create_from_theta(d, radices, perm=perm, signs=signs, theta=theta)
    xh = host_rows(rng.standard_normal((50, d)), "f32")
    gh = host_rows(rng.standard_normal((50, d)), "f32")
    grad, _, _ = _gpu_grad(plan, xh, gh, "f32")

    def loss(th_list):
        blocks = [prm.blocks_from_theta(b, th.astype(np.float64)) for b, th in zip(radices, th_list)]
        op = orc.OraclePlan(d, radices, perm, signs, [np.float32(k) for k in blocks])
        return float(np.sum(orc.forward(op, promote(xh, "f32")) * promote(gh, "f32")))

    off = 0
    for t, b in enumerate(radices):
        n = d * b
        g_theta = harp.harp_grad_theta(b, theta[t], grad[off:off + n].reshape(d // b, b, b))
        off += n
        for c, k in [(0, 0), (d // b - 1, prm.n_params(b) - 1), (3, 0)]:
            h = 1e-3
            tp = [a.astype(np.float64) for a in theta]
            tm = [a.astype(np.float64) for a in theta]
            tp[t][c, k] += h
            tm[t][c, k] -= h
            # the loss is smooth; blocks are rounded to fp32 inside loss(), hence the loose step and bound
            fd = (loss(tp) - loss(tm)) / (2 * h)
            assert abs(g_theta[c, k] - fd) <= 2e-3 * max(1.0, abs(fd)), (t, c, k, g_theta[c, k], fd)
