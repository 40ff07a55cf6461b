"""Pins of the oracle's gradient with respect to the block kernels (chain rule through
Algorithm 1).  CPU only."""
import numpy as np
import pytest

from oracle import harp_oracle as orc
from paper_2605_29843_b200 import workloads as wl

SCHEDULES = [(4,), (2, 2), (4, 3), (2, 3, 4), (8, 2, 2), (3, 5)]


def _setup(radices, seed=0, rows=6):
    spec = wl.tiny_plan(seed, radices, kind="qr", perm="random", signs=True)
    plan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(seed + 100)
    return plan, rng.standard_normal((rows, spec.d)), rng.standard_normal((rows, spec.d))


def test_single_stage_is_the_outer_product_per_block():
    """m = 1, b = d, no sign, no perm: y = x K, so dL/dK = x^T G."""
    d = 5
    rng = np.random.default_rng(1)
    K = rng.standard_normal((1, d, d))
    plan = orc.OraclePlan(d, (d,), None, None, [K])
    x, G = rng.standard_normal((7, d)), rng.standard_normal((7, d))
    (g,) = orc.grad_blocks(plan, x, G)
    assert np.allclose(g[0], x.T @ G, atol=1e-12, rtol=0)


@pytest.mark.parametrize("radices", SCHEDULES)
def test_loss_is_linear_in_each_stage_so_finite_differences_are_exact(radices):
    """L = sum(y * G) is linear in the kernels of any single stage: perturbing one entry by eps
    changes L by exactly eps times its gradient."""
    plan, x, G = _setup(radices)
    grads = orc.grad_blocks(plan, x, G)
    L0 = np.sum(orc.forward(plan, x) * G)
    rng = np.random.default_rng(9)
    for t, b in enumerate(radices):
        for _ in range(6):
            c, i, j = rng.integers(plan.d // b), rng.integers(b), rng.integers(b)
            saved = plan.blocks[t][c, i, j]
            plan.blocks[t][c, i, j] = saved + 0.5
            L1 = np.sum(orc.forward(plan, x) * G)
            plan.blocks[t][c, i, j] = saved
            assert (L1 - L0) / 0.5 == pytest.approx(grads[t][c, i, j], rel=1e-9, abs=1e-9)


@pytest.mark.parametrize("radices", SCHEDULES)
def test_euler_identity_per_stage(radices):
    """y is homogeneous of degree one in the kernels of each stage: <K_t, dL/dK_t> = L for every t."""
    plan, x, G = _setup(radices, seed=3)
    L = np.sum(orc.forward(plan, x) * G)
    for t, g in enumerate(orc.grad_blocks(plan, x, G)):
        assert np.sum(plan.blocks[t] * g) == pytest.approx(L, rel=1e-10)


def test_gradient_is_additive_over_rows_and_linear_in_g():
    plan, x, G = _setup((2, 3, 4), seed=5, rows=8)
    full = orc.grad_blocks(plan, x, G)
    a, b = orc.grad_blocks(plan, x[:3], G[:3]), orc.grad_blocks(plan, x[3:], G[3:])
    twice = orc.grad_blocks(plan, x, 2.0 * G)
    for t in range(3):
        assert np.allclose(full[t], a[t] + b[t], atol=1e-12, rtol=0)
        assert np.allclose(twice[t], 2.0 * full[t], atol=1e-12, rtol=0)


def test_a_wrong_stage_state_is_caught():
    """Using the output of a stage instead of its input in the outer product breaks the
    finite-difference pin (mutation check of the test above)."""
    plan, x, G = _setup((4, 3), seed=7)
    grads = orc.grad_blocks(plan, x, G)
    y1 = orc._stage(x * plan.signs[None, :] if plan.signs is not None else x, 4, 1, plan.blocks[0], False)
    assert not np.allclose(grads[0][0], (y1[:, :4]).T @ G[:, :4], atol=1e-6)
