"""Pins for the plan-side oracle (greedy schedule, Givens/Cayley blocks, int8 storage,
Kronecker fallback): worked examples from the paper, closed forms, Kronecker products."""
import os

import numpy as np
import pytest
import scipy.linalg

from oracle import harp_oracle as orc
from oracle import harp_params as prm

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_greedy_schedule_matches_the_papers_examples():
    for line in open(os.path.join(GOLD, "greedy_schedule.txt")):
        if line.startswith("#") or not line.strip():
            continue
        d, bb, bm, sched = line.split()
        assert prm.greedy_schedule(int(d), int(bb), int(bm)) == [int(v) for v in sched.split(",")]


@pytest.mark.parametrize("d", [2, 3, 43, 60, 11008, 14336, 28672, 8192, 12288, 22016, 97 * 8])
def test_greedy_schedule_invariants(d):
    s = prm.greedy_schedule(d)
    assert int(np.prod(s)) == d and all(b >= 2 for b in s)
    # the preferred radix comes first, then non-increasing factors up to b_max, then at most one leftover
    k = 0
    while k < len(s) and s[k] == 8:
        k += 1
    rest = s[k:]
    small = [b for b in rest if b <= 8]
    assert small == sorted(small, reverse=True)
    assert sum(1 for b in rest if b > 8) <= 1 and (not rest or all(b <= 8 for b in rest[:-1]))


def test_theta_zero_gives_the_mixer():
    for b in (2, 4, 8, 16):
        blocks = prm.blocks_from_theta(b, np.zeros((3, prm.n_params(b))))
        assert np.allclose(blocks, scipy.linalg.hadamard(b) / np.sqrt(b), atol=1e-15)
    g = np.linalg.qr(np.random.default_rng(0).standard_normal((5, 5)))[0]
    assert np.allclose(prm.blocks_from_theta(5, np.zeros((2, 10)), g), g, atol=1e-15)


def test_givens_closed_form():
    th = 0.37
    q = prm.rotation(2, np.array([th]))
    assert np.allclose(q, [[np.cos(th), -np.sin(th)], [np.sin(th), np.cos(th)]])
    x = np.array([1.0, 0.0])
    assert np.allclose(x @ q, [np.cos(th), -np.sin(th)])


def test_cayley_closed_form_and_properties():
    # b = 3 with a single non-zero entry reduces to the 2x2 Cayley map: a rotation by -2 atan(a)
    a = 0.6
    q = prm.rotation(3, np.array([a, 0.0, 0.0]))
    c, s = (1 - a * a) / (1 + a * a), 2 * a / (1 + a * a)
    assert np.allclose(q, [[c, -s, 0], [s, c, 0], [0, 0, 1]], atol=1e-15)
    rng = np.random.default_rng(1)
    for b in (3, 4, 7, 8, 16, 43):
        th = rng.normal(0, 0.3, prm.n_params(b))
        q = prm.rotation(b, th)
        A = prm.skew_from_upper(b, th)
        assert np.allclose(A, -A.T) and A[0, 1] == th[0] and A[0, b - 1] == th[b - 2] and A[1, 2] == th[b - 1]
        assert np.allclose((np.eye(b) + A) @ q, np.eye(b) - A, atol=1e-13)          # defining equation (Eq. 11)
        assert np.allclose(q.T @ q, np.eye(b), atol=1e-13) and np.isclose(np.linalg.det(q), 1.0)
        assert np.allclose(prm.rotation(b, -th), q.T, atol=1e-13)
        assert np.allclose(q, scipy.linalg.inv(np.eye(b) + A) @ (np.eye(b) - A), atol=1e-13)


@pytest.mark.parametrize("b", [2, 3, 4, 7, 8, 16])
def test_grad_theta_against_finite_differences(b):
    """L(theta) = <W, B(theta)> with a fixed W: central differences of the block reconstruction pin
    the chain rule (signs, transposes, which triangle entry belongs to which parameter)."""
    rng = np.random.default_rng(40 + b)
    npar = prm.n_params(b)
    theta = rng.normal(0, 0.4, (3, npar))
    w = rng.standard_normal((3, b, b))
    mixer = None if (b & (b - 1)) == 0 else np.linalg.qr(rng.standard_normal((b, b)))[0]
    got = prm.grad_theta(b, theta, w, mixer)
    h = 1e-6
    for c in range(3):
        for k in range(npar):
            tp, tm = theta.copy(), theta.copy()
            tp[c, k] += h
            tm[c, k] -= h
            fd = (np.sum(w * prm.blocks_from_theta(b, tp, mixer)) - np.sum(w * prm.blocks_from_theta(b, tm, mixer))) / (2 * h)
            assert abs(got[c, k] - fd) <= 1e-7 * max(1.0, abs(fd)), (c, k)


def test_grad_theta_closed_forms():
    rng = np.random.default_rng(50)
    # theta = 0, identity mixer: Q = I, dQ = -2 dA, so dL/da_ij = -2 (W_ij - W_ji)
    for b in (3, 4, 6):
        w = rng.standard_normal((1, b, b))
        got = prm.grad_theta(b, np.zeros((1, prm.n_params(b))), w, np.eye(b))[0]
        want = (-2.0 * (w[0] - w[0].T))[np.triu_indices(b, 1)]
        assert np.allclose(got, want, atol=1e-14)
    # Givens, identity mixer: L = W00 c - W01 s + W10 s + W11 c
    th, w = 0.3, rng.standard_normal((1, 2, 2))
    got = prm.grad_theta(2, np.array([[th]]), w, np.eye(2))[0, 0]
    assert np.isclose(got, -(w[0, 0, 0] + w[0, 1, 1]) * np.sin(th) + (w[0, 1, 0] - w[0, 0, 1]) * np.cos(th))
    # a loss that depends on Q only through Q^T Q (= I for every theta) has zero gradient:
    # L = ||B||_F^2 / 2 with an orthogonal mixer, dL/dB = B
    for b in (2, 5, 8):
        theta = rng.normal(0, 0.5, (4, prm.n_params(b)))
        g = np.linalg.qr(rng.standard_normal((b, b)))[0]
        blocks = prm.blocks_from_theta(b, theta, g)
        assert np.max(np.abs(prm.grad_theta(b, theta, blocks, g))) < 1e-13


def test_int8_storage_error_bound():
    rng = np.random.default_rng(2)
    theta = rng.normal(0, 0.2, (50, 28))
    theta[7] = 0.0
    q, s = prm.quantize_theta(theta)
    assert q.dtype == np.int8 and np.max(np.abs(q)) <= 127
    assert np.allclose(s, np.max(np.abs(theta), axis=1) / 127)
    back = prm.dequantize_theta(q, s)
    assert np.all(np.abs(back - theta) <= s[:, None] / 2 + 1e-15)
    assert np.all(back[7] == 0.0)


def test_kronecker_fallback_is_a_kronecker_product():
    rng = np.random.default_rng(3)
    from paper_2605_29843_b200 import workloads as wl
    # a row-permuted Hadamard matrix is still a +-1 table with H H^T = K I, but not symmetric:
    # it fixes the orientation of the Kronecker factor
    for K, hk in ((2, np.array([[1, 1], [1, -1]])), (4, scipy.linalg.hadamard(4)[[1, 3, 0, 2]]),
                  (8, scipy.linalg.hadamard(8)[[5, 0, 7, 2, 1, 6, 3, 4]])):
        assert np.array_equal(hk @ hk.T, K * np.eye(K)) and (K == 2 or not np.array_equal(hk, hk.T))
        radices = (4, 2)
        n2 = 8
        blocks = [wl.qr_orthogonal(rng, n2 // b, b) for b in radices]
        t_small = orc.dense(orc.OraclePlan(n2, radices, None, None, blocks))
        rd, bd = prm.kronecker_stage_blocks(n2, radices, blocks, K, hk)
        t_big = orc.dense(orc.OraclePlan(K * n2, rd, None, None, bd))
        assert np.allclose(t_big, np.kron(hk / np.sqrt(K), t_small), atol=1e-13)
