"""CPU oracle for the diagnostics of a processed layer.  TEST INFRASTRUCTURE ONLY: nothing in
the product path may import this file (tests, the smoke check and the CPU-baseline leg of the
benchmark may).  Plain numpy in fp64, each function the definition it cites, written out.

Pins (tests/test_diagnostics_oracle.py): closed forms for constant, one-hot and identity
matrices, the bounds 1 <= mu_W <= sqrt(mn), invariance of the Frobenius norm under orthogonal
maps, brute-force loops on tiny inputs, and scaling laws of every quantity.
"""
from __future__ import annotations

import numpy as np


def weight_incoherence(A) -> float:
    """Eq. 4: mu_W(A) = sqrt(m n) * max_ij |A_ij| / ||A||_F."""
    A = np.asarray(A, dtype=np.float64)
    m, n = A.shape
    fro = np.sqrt(np.sum(A * A))
    if fro == 0.0:
        return 0.0
    return float(np.sqrt(m * n) * np.max(np.abs(A)) / fro)


def offblock_energy(H, block: int) -> float:
    """Eq. 15: (1/n^2) * sum over block pairs p != q of ||H_pq||_F^2, the blocks being
    consecutive runs of `block` coordinates (the last run may be shorter)."""
    H = np.asarray(H, dtype=np.float64)
    n = H.shape[0]
    assert H.shape == (n, n) and 1 <= block <= n
    total = 0.0
    starts = list(range(0, n, block))
    for p in starts:
        for q in starts:
            if p != q:
                blk = H[p:p + block, q:q + block]
                total += float(np.sum(blk * blk))
    return total / (n * n)


def diag_weighted_error(Wt, Wq, H) -> float:
    """Eq. 14: (1/(d_out d_in)) * sum_ij Delta_ij^2 * wbar_j with Delta = Wt - Wq,
    w_j = |H_jj| and wbar = w / mean(w)."""
    Wt = np.asarray(Wt, dtype=np.float64)
    Wq = np.asarray(Wq, dtype=np.float64)
    H = np.asarray(H, dtype=np.float64)
    d_out, d_in = Wt.shape
    w = np.abs(np.diag(H))
    mean = np.mean(w)
    if mean == 0.0:
        return 0.0
    wbar = w / mean
    delta = Wt - Wq
    return float(np.sum(delta * delta * wbar[None, :]) / (d_out * d_in))
