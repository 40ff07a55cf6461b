"""Pins for the CPU oracle: every check here compares the oracle with something
built another way -- dense matrices assembled from the index formula, Kronecker
products, scipy's Hadamard matrix, a plain matrix product, or values written in
the paper (tests/golden)."""
import os

import numpy as np
import pytest
import scipy.linalg

from oracle import harp_oracle as orc
from paper_2605_29843_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")

TINY = [(2, 2, 2), (4, 4), (2, 3), (7, 2), (3, 5, 2), (16, 4), (43,), (2, 2, 7), (8, 8), (5, 4, 3)]


# ---------- independent dense construction (index formula of Lemma 1) ----------

def dense_stage(d, b, s, K):
    """Row-acting matrix of one stage: M[p_in, p_out] = K[c][i][j] for
    p_in = alpha*b*s + i*s + beta, p_out = alpha*b*s + j*s + beta, c = alpha*s + beta."""
    M = np.zeros((d, d))
    g = d // (b * s)
    for alpha in range(g):
        for beta in range(s):
            c = alpha * s + beta
            for i in range(b):
                for j in range(b):
                    M[alpha * b * s + i * s + beta, alpha * b * s + j * s + beta] = K[c][i][j]
    return M


def dense_Q(spec):
    d = spec.d
    Q = np.eye(d)
    if spec.signs is not None:
        Q = Q @ np.diag(spec.signs.astype(np.float64))
    if spec.perm is not None:
        P = np.zeros((d, d))
        for i in range(d):
            P[spec.perm[i], i] = 1.0          # (u P)_i = u_{perm[i]}
        Q = Q @ P
    s = 1
    for t, b in enumerate(spec.radices):
        Q = Q @ dense_stage(d, b, s, spec.blocks[t].astype(np.float64))
        s *= b
    return Q


@pytest.mark.parametrize("radices", TINY)
def test_forward_and_transpose_equal_dense_product(radices):
    spec = wl.tiny_plan(7, radices, kind="qr", perm="random", signs=True)
    plan = orc.OraclePlan.from_spec(spec)
    Q = dense_Q(spec)
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, spec.d))
    assert np.allclose(orc.forward(plan, x), x @ Q, atol=1e-12, rtol=0)
    assert np.allclose(orc.transpose(plan, x), x @ Q.T, atol=1e-12, rtol=0)
    assert np.allclose(orc.dense(plan), Q, atol=1e-12, rtol=0)


def test_passes_compose_as_a_product_of_dense_matrices():
    """Several passes: forward is x Q_0 Q_1 Q_2 with each Q_k built independently from its own
    stages; the transpose is the inverse, applied in the opposite order."""
    specs = [wl.tiny_plan(3, (4, 2, 3), kind="qr", perm="random", signs=True),
             wl.tiny_plan(4, (3, 8), kind="qr", perm="identity", signs=False),
             wl.tiny_plan(5, (2, 2, 6), kind="qr", perm="random", signs=False)]
    plans = [orc.OraclePlan.from_spec(sp) for sp in specs]
    Qs = [dense_Q(sp) for sp in specs]
    x = np.random.default_rng(2).standard_normal((4, 24))
    assert np.allclose(orc.forward_passes(plans, x), x @ Qs[0] @ Qs[1] @ Qs[2], atol=1e-12, rtol=0)
    assert np.allclose(orc.transpose_passes(plans, x), x @ Qs[2].T @ Qs[1].T @ Qs[0].T, atol=1e-12, rtol=0)
    # (the blocks are orthogonal to fp32 rounding only)
    assert np.allclose(orc.transpose_passes(plans, orc.forward_passes(plans, x)), x, atol=1e-5, rtol=0)
    # the order matters: the passes do not commute
    assert not np.allclose(orc.forward_passes(plans[::-1], x), orc.forward_passes(plans, x), atol=1e-6)
    # one pass is the plain apply
    assert np.array_equal(orc.forward_passes(plans[:1], x), orc.forward(plans[0], x))


@pytest.mark.parametrize("radices", TINY)
def test_orthogonality_dense(radices):
    plan = orc.OraclePlan.from_spec(wl.tiny_plan(3, radices))
    Q = orc.dense(plan)
    assert np.max(np.abs(Q.T @ Q - np.eye(plan.d))) < 1e-6   # blocks are fp32-rounded
    spec64 = wl.tiny_plan(3, radices)
    rng = np.random.default_rng(0)
    spec64.blocks = [wl.qr_orthogonal(rng, spec64.d // b, b) for b in radices]   # fp64 blocks
    Q = orc.dense(orc.OraclePlan.from_spec(spec64))
    assert np.max(np.abs(Q.T @ Q - np.eye(plan.d))) < 1e-12


@pytest.mark.parametrize("radices", [(2, 2, 2), (4, 4), (3, 5, 2), (2, 4, 3)])
def test_stage_is_kronecker_product_for_equal_blocks(radices):
    """S_t = I_g (x) B (x) I_s when all blocks of the stage are the same (Lemma 1)."""
    d = int(np.prod(radices))
    rng = np.random.default_rng(5)
    mats = [wl.qr_orthogonal(rng, 1, b)[0] for b in radices]
    blocks = [np.broadcast_to(B, (d // B.shape[0],) + B.shape).copy() for B in mats]
    plan = orc.OraclePlan(d, radices, None, None, blocks)
    Q = np.eye(d)
    s = 1
    for B in mats:
        b = B.shape[0]
        Q = Q @ np.kron(np.kron(np.eye(d // (b * s)), B), np.eye(s))
        s *= b
    assert np.allclose(orc.dense(plan), Q, atol=1e-13, rtol=0)
    # product of Kronecker stages = B_{m-1} (x) ... (x) B_0
    full = np.eye(1)
    for B in mats:
        full = np.kron(B, full)
    assert np.allclose(orc.dense(plan), full, atol=1e-13, rtol=0)


def test_single_stage_is_a_plain_matrix_product():
    """m = 1, b = d: the transform is x @ K (fixes the orientation out_j = sum_i in_i K[i][j])."""
    rng = np.random.default_rng(2)
    K = rng.standard_normal((1, 11, 11))
    plan = orc.OraclePlan(11, (11,), None, None, [K])
    x = rng.standard_normal((4, 11))
    assert np.allclose(orc.forward(plan, x), x @ K[0], atol=1e-13, rtol=0)
    assert np.allclose(orc.transpose(plan, x), x @ K[0].T, atol=1e-13, rtol=0)


def test_block_index_is_alpha_times_s_plus_beta():
    """Only block c = alpha*s+beta of a stage may touch coordinates {alpha b s + r s + beta}."""
    d, radices = 24, (2, 3, 4)
    strides = (1, 2, 6)
    for t, (b, s) in enumerate(zip(radices, strides)):
        g = d // (b * s)
        for c in range(d // b):
            blocks = [np.broadcast_to(np.eye(bb), (d // bb, bb, bb)).copy() for bb in radices]
            blocks[t][c] = 2.0 * np.eye(b)
            Q = orc.dense(orc.OraclePlan(d, radices, None, None, blocks))
            alpha, beta = divmod(c, s)
            assert alpha < g
            want = np.ones(d)
            want[[alpha * b * s + r * s + beta for r in range(b)]] = 2.0
            assert np.array_equal(np.diag(Q), want) and np.count_nonzero(Q) == d


# ---------- the paper's worked index example ----------

def _golden_groups():
    groups, cur = {}, None
    for line in open(os.path.join(GOLD, "index_example_d16_b4.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("stage"):
            cur = int(line.split()[1])
            groups[cur] = []
        else:
            groups[cur].append([int(v) for v in line.split()])
    return groups


def test_index_example_d16_b4():
    groups = _golden_groups()
    rng = np.random.default_rng(9)
    for t in (0, 1):
        blocks = [np.broadcast_to(np.eye(4), (4, 4, 4)).copy() for _ in range(2)]
        blocks[t] = rng.uniform(1.0, 2.0, size=(4, 4, 4))        # dense, no zero entries
        Q = orc.dense(orc.OraclePlan(16, (4, 4), None, None, blocks))
        pattern = np.zeros((16, 16), dtype=bool)
        for grp in groups[t]:
            pattern[np.ix_(grp, grp)] = True
        assert np.array_equal(Q != 0.0, pattern)


# ---------- exact initialisation recovers the randomised Hadamard transform ----------

def _sylvester_from_recursion(d):
    h = np.ones((1, 1))
    while h.shape[0] < d:
        h = np.block([[h, h], [h, -h]])
    return h / np.sqrt(d)


def test_sylvester_golden_and_scipy():
    h4 = np.loadtxt(os.path.join(GOLD, "sylvester_recursion.txt"))
    assert np.array_equal(_sylvester_from_recursion(4) * 2.0, h4)
    assert np.array_equal(scipy.linalg.hadamard(64) / 8.0, _sylvester_from_recursion(64))


@pytest.mark.parametrize("radices", [(2, 2, 2), (2,) * 6, (4, 4, 4), (8, 8), (16, 16, 8, 2), (2, 16, 4),
                                     (2,) * 11, (4,) * 6])
def test_theta_zero_is_the_hadamard_transform(radices):
    d = int(np.prod(radices))
    H = scipy.linalg.hadamard(d).astype(np.float64) / np.sqrt(d)
    rng = np.random.default_rng(3)
    signs = wl.rademacher(rng, d)
    blocks = [np.broadcast_to(scipy.linalg.hadamard(b) / np.sqrt(b), (d // b, b, b)).copy() for b in radices]
    x = rng.standard_normal((3, d))
    # no permutation: T(0) = H_d exactly for every power-of-two schedule
    y = orc.forward(orc.OraclePlan(d, radices, None, signs, blocks), x)
    assert np.allclose(y, (x * signs) @ H, atol=1e-12, rtol=0)
    # with the digit-reversal permutation: gather, then H_d; H_d is invariant under it
    perm = wl.digit_reversal_perm(radices)
    y = orc.forward(orc.OraclePlan(d, radices, perm, signs, blocks), x)
    assert np.allclose(y, (x * signs)[:, perm] @ H, atol=1e-12, rtol=0)
    if len(set(radices)) == 1:
        assert np.allclose(y, ((x * signs) @ H)[:, perm], atol=1e-12, rtol=0)


def test_generator_theta_zero_blocks_are_hadamard():
    spec = wl.make_plan(0, 64, (2, 4, 8), "hadamard", signs=False)
    for b, k in zip(spec.radices, spec.blocks):
        assert np.allclose(k, scipy.linalg.hadamard(b) / np.sqrt(b), atol=1e-7)
    assert np.allclose(wl.givens_times_h2(np.zeros(1))[0], scipy.linalg.hadamard(2) / np.sqrt(2))
    assert np.allclose(wl.expm_skew(np.zeros((1, 4, 4)))[0], np.eye(4))


# ---------- permutation and signs are exact ----------

@pytest.mark.parametrize("radices", [(2, 2, 2), (3, 5, 2), (4, 4, 4)])
def test_identity_blocks_give_exact_sign_and_gather(radices):
    spec = wl.tiny_plan(11, radices, kind="identity", perm="random", signs=True)
    plan = orc.OraclePlan.from_spec(spec)
    x = np.random.default_rng(4).standard_normal((6, spec.d))
    y = orc.forward(plan, x)
    assert np.array_equal(y, (x * spec.signs)[:, spec.perm])
    assert np.array_equal(orc.transpose(plan, y), x)


def test_digit_reversal_perm_properties():
    p = wl.digit_reversal_perm((4,) * 6)
    assert sorted(p.tolist()) == list(range(4096))
    assert np.array_equal(p[p], np.arange(4096))                 # involution for equal radices
    p = wl.digit_reversal_perm((2, 3, 4))                        # i = i0 + 2 i1 + 6 i2 -> i0*12 + i1*4 + i2
    assert p[1] == 12 and p[2] == 4 and p[6] == 1
    assert sorted(p.tolist()) == list(range(24))


# ---------- round trip, norms, two-sided ----------

@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_round_trip_and_norm_at_config_sizes(cfg):
    w = wl.config(cfg, n_rows=4)
    spec = w.plans["q"]
    plan = orc.OraclePlan.from_spec(spec)
    x = w.data["x"].rows_f64(0, 4)
    y = orc.forward(plan, x)
    # blocks are orthogonal to fp32 rounding (~1e-7 per stage)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=2e-6)
    back = orc.transpose(plan, y)
    assert orc.rel_err_rows(back, x) < 2e-6
    for t, b in enumerate(spec.radices):
        k = spec.blocks[t].astype(np.float64)
        assert np.max(np.abs(np.swapaxes(k, 1, 2) @ k - np.eye(b))) < 1e-6


def test_round_trip_is_exact_for_exactly_orthogonal_blocks():
    rng = np.random.default_rng(8)
    radices = (4, 3, 8, 5)
    d = 480
    blocks = [wl.qr_orthogonal(rng, d // b, b) for b in radices]           # fp64
    plan = orc.OraclePlan(d, radices, rng.permutation(d), wl.rademacher(rng, d), blocks)
    x = rng.standard_normal((7, d))
    y = orc.forward(plan, x)
    assert np.allclose(orc.transpose(plan, y), x, atol=1e-13, rtol=0)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-13)


def test_two_sided_equals_dense_and_keeps_the_layer_function():
    p_out = wl.tiny_plan(21, (3, 4), kind="qr", perm="random")
    p_in = wl.tiny_plan(22, (2, 5, 2), kind="qr", perm="random")
    po, pi = orc.OraclePlan.from_spec(p_out), orc.OraclePlan.from_spec(p_in)
    rng = np.random.default_rng(6)
    W = rng.standard_normal((12, 20))
    Wt = orc.two_sided(po, pi, W)
    assert np.allclose(Wt, dense_Q(p_out).T @ W @ dense_Q(p_in), atol=1e-12, rtol=0)
    assert np.isclose(np.linalg.norm(Wt), np.linalg.norm(W), rtol=1e-6)
    # y = x W^T is recovered as transpose_out(forward_in(x) W~^T)
    x = rng.standard_normal((3, 20))
    y = orc.transpose(po, orc.forward(pi, x) @ Wt.T)
    assert np.allclose(y, x @ W.T, atol=1e-5, rtol=0)


def test_parameter_count_of_the_generator_matches_eq13():
    for line in open(os.path.join(GOLD, "param_count.txt")):
        if line.startswith("#") or not line.strip():
            continue
        d, sched, total = line.split()
        radices = tuple(int(v) for v in sched.split(","))
        spec = wl.make_plan(0, int(d), radices, "identity", signs=False)
        dof = sum(k.shape[0] * b * (b - 1) // 2 for b, k in zip(radices, spec.blocks))
        assert dof == int(total)


def test_plan_validation():
    eye = [np.broadcast_to(np.eye(2), (2, 2, 2)).copy()] * 2
    with pytest.raises(ValueError):
        orc.OraclePlan(5, (2, 2), None, None, eye)
    with pytest.raises(ValueError):
        orc.OraclePlan(4, (2, 2), np.array([0, 1, 1, 3]), None, eye)
    with pytest.raises(ValueError):
        orc.OraclePlan(4, (2, 2), None, np.array([1, -1, 0, 1]), eye)


# ---------- planted mistakes must be caught by the pins above ----------

def test_pins_catch_a_transposed_block_and_a_wrong_block_index():
    spec = wl.tiny_plan(7, (3, 5, 2), kind="qr", perm="random", signs=True)
    Q = dense_Q(spec)
    x = np.random.default_rng(1).standard_normal((5, spec.d))
    bad = wl.tiny_plan(7, (3, 5, 2), kind="qr", perm="random", signs=True)
    bad.blocks = [np.swapaxes(k, 1, 2).copy() for k in bad.blocks]            # transposed operand
    assert not np.allclose(orc.forward(orc.OraclePlan.from_spec(bad), x), x @ Q, atol=1e-6)
    bad = wl.tiny_plan(7, (3, 5, 2), kind="qr", perm="random", signs=True)
    bad.blocks[1] = bad.blocks[1][::-1].copy()                                # wrong block order
    assert not np.allclose(orc.forward(orc.OraclePlan.from_spec(bad), x), x @ Q, atol=1e-6)
