"""CPU oracle for the plan-side helpers -- TEST INFRASTRUCTURE, not the product.

* greedy_schedule      : Algorithm 2 (greedy Mixed-Radix schedule, preferred radix first).
* blocks_from_theta    : block kernels B = Q(theta) G_b (Eq. 9) with Q a Givens rotation for
                         b = 2 (Eq. 10) and the Cayley map Q = (I + A)^{-1} (I - A) of a
                         skew-symmetric A for b > 2 (Eq. 11); A is given by its strict upper
                         triangle (row-major, i < j), A_ji = -A_ij.
* grad_theta           : chain rule from dL/dB back to theta through Eq. 9-11.
* dequantize_theta     : int8 storage (appendix "Int8 storage of HARP parameters"):
                         a ~ s * q with one scale per block.
* quantize_theta       : s = max|a| / 127, q = round(a / s).
* kronecker_spec       : Kronecker fallback T_d = (H~_K / sqrt K) (x) T_{n2} (Eq. 12) written as
                         a stage list: the stages of T_{n2}, replicated for each of the K rows,
                         then one radix-K stage of stride n2 whose blocks all equal H~_K/sqrt K.
Plain numpy, fp64.  Pinned in tests/test_params_oracle.py by the paper's worked schedules,
closed forms and Kronecker products.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np


def greedy_schedule(d: int, b_base: int = 8, b_max: int = 8) -> List[int]:
    """Algorithm 2 as a recurrence on the part of d not yet factored: the next stage takes the preferred
    radix b_base while it divides what is left, otherwise the largest divisor of what is left that does
    not exceed b_max, and a remainder without such a divisor becomes the last stage itself."""
    if d < 2:
        raise ValueError("d >= 2 required")

    def next_radix(rest: int, base_allowed: bool):
        if base_allowed and rest % b_base == 0:
            return b_base, True
        for f in range(min(b_max, rest), 1, -1):
            if rest % f == 0:
                return f, False
        return rest, False

    out, rest, base_allowed = [], d, True
    while rest > 1:
        b, base_allowed = next_radix(rest, base_allowed)
        out.append(b)
        rest //= b
    return out


def sylvester(b: int) -> np.ndarray:
    h = np.ones((1, 1))
    while h.shape[0] < b:
        h = np.block([[h, h], [h, -h]])
    return h / np.sqrt(b)


def skew_from_upper(b: int, upper: np.ndarray) -> np.ndarray:
    a = np.zeros((b, b))
    a[np.triu_indices(b, 1)] = upper
    return a - a.T


def rotation(b: int, theta: np.ndarray) -> np.ndarray:
    """Q(theta): Givens for b = 2 (theta = one angle), Cayley otherwise (theta = upper triangle of A)."""
    if b == 2:
        c, s = np.cos(theta[0]), np.sin(theta[0])
        return np.array([[c, -s], [s, c]])
    a = skew_from_upper(b, theta)
    eye = np.eye(b)
    return np.linalg.solve(eye + a, eye - a)


def n_params(b: int) -> int:
    return 1 if b == 2 else b * (b - 1) // 2


def blocks_from_theta(b: int, theta: np.ndarray, mixer: Optional[np.ndarray] = None) -> np.ndarray:
    """theta[n_blocks, n_params(b)] -> blocks[n_blocks, b, b] = Q(theta_c) G_b."""
    g = sylvester(b) if mixer is None else np.asarray(mixer, dtype=np.float64)
    theta = np.asarray(theta, dtype=np.float64).reshape(-1, n_params(b))
    return np.stack([rotation(b, th) @ g for th in theta])


def grad_theta(b: int, theta: np.ndarray, grad_blocks: np.ndarray, mixer: Optional[np.ndarray] = None) -> np.ndarray:
    """dL/dtheta[n_blocks, n_params(b)] from dL/dB[n_blocks, b, b] for B = Q(theta) G_b (Eq. 9-11).

    D = dL/dQ = (dL/dB) G^T.  Givens (Eq. 10): dL/dtheta = <D, dQ/dtheta>.  Cayley (Eq. 11):
    differentiating (I + A) Q = I - A gives dQ = -(I + A)^{-1} dA (Q + I), so
    dL/dA = -(I + A)^{-T} D (Q + I)^T, and the entry of the pair i < j is (dL/dA)_ij - (dL/dA)_ji
    because A_ji = -A_ij."""
    g = sylvester(b) if mixer is None else np.asarray(mixer, dtype=np.float64)
    theta = np.asarray(theta, dtype=np.float64).reshape(-1, n_params(b))
    gb = np.asarray(grad_blocks, dtype=np.float64).reshape(-1, b, b)
    out = np.empty_like(theta)
    eye = np.eye(b)
    iu = np.triu_indices(b, 1)
    for c, th in enumerate(theta):
        dq = gb[c] @ g.T
        if b == 2:
            cs, sn = np.cos(th[0]), np.sin(th[0])
            out[c, 0] = np.sum(dq * np.array([[-sn, -cs], [cs, -sn]]))
            continue
        a = skew_from_upper(b, th)
        q = np.linalg.solve(eye + a, eye - a)
        da = -np.linalg.solve((eye + a).T, dq) @ (q + eye).T
        out[c] = (da - da.T)[iu]
    return out


def quantize_theta(theta: np.ndarray):
    theta = np.asarray(theta, dtype=np.float64)
    s = np.max(np.abs(theta), axis=1) / 127.0
    safe = np.where(s == 0.0, 1.0, s)
    q = np.rint(theta / safe[:, None]).astype(np.int8)
    return q, s


def dequantize_theta(q: np.ndarray, s: np.ndarray) -> np.ndarray:
    return q.astype(np.float64) * np.asarray(s, dtype=np.float64)[:, None]


def kronecker_stage_blocks(n2: int, radices: Sequence[int], blocks_n2: Sequence[np.ndarray], K: int, hk: np.ndarray):
    """Returns (radices_d, blocks_d) of the d = K*n2 plan equal to (H~_K/sqrt K) (x) T_{n2}."""
    d = K * n2
    out_r, out_b = [], []
    s = 1
    for b, blk in zip(radices, blocks_n2):
        blk = np.asarray(blk, dtype=np.float64)          # [n2/b, b, b], block c = alpha*s + beta inside one row
        g_small = n2 // (b * s)
        big = np.empty((d // b, b, b))
        # full-size block index: alpha_d = k*g_small + alpha  (the K rows are the slowest index)
        for k in range(K):
            for alpha in range(g_small):
                for beta in range(s):
                    big[(k * g_small + alpha) * s + beta] = blk[alpha * s + beta]
        out_r.append(b)
        out_b.append(big)
        s *= b
    hk = np.asarray(hk, dtype=np.float64) / np.sqrt(K)
    out_r.append(K)
    out_b.append(np.broadcast_to(hk, (n2, K, K)).copy())
    return out_r, out_b
