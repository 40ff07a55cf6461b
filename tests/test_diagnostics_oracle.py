"""Pins of the diagnostics oracle (Eq. 4, Eq. 14, Eq. 15) against closed forms, bounds,
invariances and brute force.  CPU only."""
import numpy as np
import pytest

from oracle import harp_diagnostics as od


def test_mu_w_closed_forms():
    # constant matrix: every entry carries the same share -> mu = 1, the minimum
    assert od.weight_incoherence(np.full((7, 5), -3.0)) == pytest.approx(1.0, rel=1e-14)
    # a single non-zero entry: all the mass on one coordinate -> mu = sqrt(mn), the maximum
    A = np.zeros((6, 11)); A[2, 9] = 0.25
    assert od.weight_incoherence(A) == pytest.approx(np.sqrt(66.0), rel=1e-14)
    # identity n x n: max 1, ||I||_F = sqrt(n) -> mu = n / sqrt(n) = sqrt(n)
    assert od.weight_incoherence(np.eye(9)) == pytest.approx(3.0, rel=1e-14)
    assert od.weight_incoherence(np.zeros((3, 3))) == 0.0


def test_mu_w_bounds_scale_and_transpose():
    rng = np.random.default_rng(5)
    A = rng.standard_t(3, size=(40, 24))
    mu = od.weight_incoherence(A)
    assert 1.0 <= mu <= np.sqrt(A.size)
    assert od.weight_incoherence(-17.5 * A) == pytest.approx(mu, rel=1e-13)      # scale invariant
    assert od.weight_incoherence(A.T) == pytest.approx(mu, rel=1e-13)
    # brute force
    mx, ss = 0.0, 0.0
    for v in A.ravel():
        mx = max(mx, abs(v)); ss += v * v
    assert mu == pytest.approx(np.sqrt(A.size) * mx / np.sqrt(ss), rel=1e-13)


def test_mu_w_drops_under_a_hadamard_rotation_of_an_outlier():
    # one outlier channel spread by an orthonormal Hadamard: the Frobenius norm is kept, the max drops
    n = 16
    H = np.array([[(-1.0) ** bin(i & j).count("1") for j in range(n)] for i in range(n)]) / 4.0
    A = np.zeros((4, n)); A[:, 3] = 8.0
    assert od.weight_incoherence(A) == pytest.approx(np.sqrt(4 * n) * 8.0 / 16.0)
    B = A @ H
    assert np.sum(B * B) == pytest.approx(np.sum(A * A), rel=1e-13)
    assert od.weight_incoherence(B) == pytest.approx(1.0, rel=1e-13)            # all |entries| equal 2


def test_offblock_closed_forms():
    n, g = 12, 4
    assert od.offblock_energy(np.eye(n), g) == 0.0
    # all-ones: n^2 entries, n*g of them inside the diagonal blocks
    assert od.offblock_energy(np.ones((n, n)), g) == pytest.approx((n * n - n * g) / (n * n))
    # block = n: one block, nothing off it; block = 1: everything but the diagonal
    M = np.arange(36.0).reshape(6, 6)
    assert od.offblock_energy(M, 6) == 0.0
    assert od.offblock_energy(M, 1) == pytest.approx((np.sum(M * M) - np.sum(np.diag(M) ** 2)) / 36.0)
    # block-diagonal input has no off-block energy
    B = np.zeros((8, 8)); B[:4, :4] = 2.0; B[4:, 4:] = -1.0
    assert od.offblock_energy(B, 4) == 0.0
    assert od.offblock_energy(B, 2) == pytest.approx((8 * 4.0 + 8 * 1.0) / 64.0)


def test_offblock_ragged_last_block_and_brute_force():
    rng = np.random.default_rng(11)
    n, g = 10, 4                                   # blocks [0,4) [4,8) [8,10)
    M = rng.standard_normal((n, n))
    brute = 0.0
    for i in range(n):
        for j in range(n):
            if i // g != j // g:
                brute += M[i, j] ** 2
    assert od.offblock_energy(M, g) == pytest.approx(brute / n ** 2, rel=1e-13)
    assert od.offblock_energy(3.0 * M, g) == pytest.approx(9.0 * brute / n ** 2, rel=1e-13)   # quadratic in H


def test_diag_weighted_error_closed_forms():
    rng = np.random.default_rng(3)
    Wt = rng.standard_normal((5, 8)); Wq = Wt + 0.5
    # equal weights: wbar = 1 -> plain mean squared error
    assert od.diag_weighted_error(Wt, Wq, 7.0 * np.eye(8)) == pytest.approx(0.25, rel=1e-13)
    # all weight on one column: wbar_j = d_in there
    H = np.zeros((8, 8)); H[2, 2] = -4.0          # the absolute value of the diagonal is used
    Wq2 = Wt.copy(); Wq2[:, 2] += 2.0; Wq2[:, 5] += 100.0
    assert od.diag_weighted_error(Wt, Wq2, H) == pytest.approx(8 * 5 * 4.0 / 40.0, rel=1e-13)
    assert od.diag_weighted_error(Wt, Wt, H) == 0.0
    assert od.diag_weighted_error(Wt, Wq, np.zeros((8, 8))) == 0.0


def test_diag_weighted_error_brute_force_and_scale_invariance_in_h():
    rng = np.random.default_rng(4)
    Wt = rng.standard_normal((6, 9)); Wq = np.round(Wt * 2) / 2
    X = rng.standard_normal((30, 9)); H = X.T @ X
    w = [abs(H[j, j]) for j in range(9)]
    mean = sum(w) / 9
    brute = sum((Wt[i, j] - Wq[i, j]) ** 2 * w[j] / mean for i in range(6) for j in range(9)) / 54
    assert od.diag_weighted_error(Wt, Wq, H) == pytest.approx(brute, rel=1e-13)
    assert od.diag_weighted_error(Wt, Wq, 123.0 * H) == pytest.approx(brute, rel=1e-13)   # wbar is normalised
