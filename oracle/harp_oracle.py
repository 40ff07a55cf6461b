"""CPU oracle for the HARP apply path -- TEST INFRASTRUCTURE, not the product.

Plain, slow, fp64 numpy.  Only tests, the smoke check and the benchmark's CPU
baseline may import this module; the CUDA library never does, and this module
imports nothing from the CUDA package.

What it computes (row-vector convention of Algorithm 1, y = x T(Theta)):

    forward(x)   = x . D_s . Pi . M_0 . M_1 ... M_{m-1}
    transpose(y) = y . M_{m-1}^T ... M_0^T . Pi^T . D_s

* D_s   : the Rademacher sign diagonal (Section "HARP processors", Assumption 1(d)):
          u_i = s_i x_i.
* Pi    : the fixed permutation, applied as a gather v_i = u_{perm[i]}.
* M_t   : stage t of Eq. 7 acting on a row vector.  Following Algorithm 1 the row is
          reshaped to (g, b_t, s_t) with s_t = prod_{j<t} b_j and g = d/(b_t s_t)
          (the flattening X[alpha, r, beta] = x[alpha b s + r s + beta] of Lemma 1),
          transposed to (g, s_t, b_t), each length-b_t group is multiplied on the
          right by its own kernel K_t[alpha, beta] (K_t viewed as g x s x b x b), and
          the transpose/reshape is inverted.  Stage 0 is applied first (Eq. 8).

Two-sided processing (Section "Incoherence processing"): W~ = U^T W V with
U = Q_out, V = Q_in, i.e. every row of W goes through forward_in and every column
through forward_out.

Readings taken where the paper leaves a choice open: a block acts as
out_j = sum_i in_i K[i][j]; block index c = alpha*s_t + beta; signs act on the
input coordinate, before the gather.

Every public function is pinned by tests against dense matrices built from the
index formula, Kronecker products, the Sylvester Hadamard matrix and brute force.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np


class OraclePlan:
    """fp64 copy of a processor description (schedule, perm, signs, block kernels)."""

    def __init__(self, d: int, radices: Sequence[int], perm: Optional[np.ndarray],
                 signs: Optional[np.ndarray], blocks: List[np.ndarray]):
        self.d = int(d)
        self.radices = [int(b) for b in radices]
        prod = 1
        for b in self.radices:
            if b < 2:
                raise ValueError("radix < 2")
            prod *= b
        if prod != self.d:
            raise ValueError("prod(radices) != d")                      # Eq. 6
        self.perm = None if perm is None else np.asarray(perm, dtype=np.int64)
        if self.perm is not None and sorted(self.perm.tolist()) != list(range(self.d)):
            raise ValueError("perm is not a bijection")
        self.signs = None if signs is None else np.asarray(signs, dtype=np.float64)
        if self.signs is not None and not np.all(np.abs(self.signs) == 1.0):
            raise ValueError("signs not in {+1,-1}")
        self.blocks = []
        for t, b in enumerate(self.radices):
            k = np.asarray(blocks[t], dtype=np.float64)
            if k.shape != (self.d // b, b, b):
                raise ValueError(f"stage {t}: blocks must be [d/b, b, b]")
            self.blocks.append(k)

    @classmethod
    def from_spec(cls, spec) -> "OraclePlan":
        return cls(spec.d, spec.radices, spec.perm, spec.signs, spec.blocks)


def _stage(y: np.ndarray, b: int, s: int, k: np.ndarray, transposed: bool) -> np.ndarray:
    """One stride stage of Algorithm 1 on a batch y[B, d]."""
    n, d = y.shape
    g = d // (b * s)
    yh = y.reshape(n, g, b, s).transpose(0, 1, 3, 2)          # B x g x s x b
    kv = k.reshape(g, s, b, b)                                 # view of K_t
    if transposed:
        kv = kv.transpose(0, 1, 3, 2)
    zh = np.einsum("ngsi,gsij->ngsj", yh, kv)                  # multiply along last dim
    return zh.transpose(0, 1, 3, 2).reshape(n, d)              # invert transpose/reshape


def forward(plan: OraclePlan, x: np.ndarray) -> np.ndarray:
    """y = x . D_s . Pi . T  for a batch of rows x[B, d] (fp64)."""
    y = np.array(x, dtype=np.float64, ndmin=2)
    if plan.signs is not None:
        y = y * plan.signs[None, :]
    if plan.perm is not None:
        y = y[:, plan.perm]
    s = 1
    for t, b in enumerate(plan.radices):                       # stage 0 first (Eq. 8)
        y = _stage(y, b, s, plan.blocks[t], transposed=False)
        s *= b
    return y


def transpose(plan: OraclePlan, y: np.ndarray) -> np.ndarray:
    """x = y . T^T . Pi^T . D_s : the inverse of forward for orthogonal blocks."""
    v = np.array(y, dtype=np.float64, ndmin=2)
    strides = []
    s = 1
    for b in plan.radices:
        strides.append(s)
        s *= b
    for t in range(len(plan.radices) - 1, -1, -1):
        v = _stage(v, plan.radices[t], strides[t], plan.blocks[t], transposed=True)
    if plan.perm is not None:
        w = np.empty_like(v)
        w[:, plan.perm] = v                                     # scatter: w[perm[i]] = v[i]
        v = w
    if plan.signs is not None:
        v = v * plan.signs[None, :]
    return v


def two_sided(plan_out: OraclePlan, plan_in: OraclePlan, w: np.ndarray) -> np.ndarray:
    """W~ = Q_out^T W Q_in for W[d_out, d_in]."""
    w = np.asarray(w, dtype=np.float64)
    assert w.shape == (plan_out.d, plan_in.d)
    rows_done = forward(plan_in, w)                             # each row . Q_in
    return forward(plan_out, rows_done.T).T                     # each column . Q_out


def grad_blocks(plan: OraclePlan, x: np.ndarray, gy: np.ndarray) -> List[np.ndarray]:
    """dL/dK_t for y = forward(x) and G = dL/dy (chain rule through Algorithm 1):
    g_m = G, g_t = g_{t+1} M_t^T, dL/dK_t[c][i][j] = sum_rows v_t[base_c + i s_t] g_{t+1}[base_c + j s_t],
    with v_t the input of stage t.  Returns one array [D_t][b_t][b_t] per stage."""
    v = np.array(x, dtype=np.float64, ndmin=2)
    if plan.signs is not None:
        v = v * plan.signs[None, :]
    if plan.perm is not None:
        v = v[:, plan.perm]
    n = v.shape[0]
    states, strides = [], []
    s = 1
    for t, b in enumerate(plan.radices):
        states.append(v)                                       # v_t: what stage t reads
        strides.append(s)
        v = _stage(v, b, s, plan.blocks[t], transposed=False)
        s *= b
    g = np.array(gy, dtype=np.float64, ndmin=2)
    grads: List[np.ndarray] = [np.zeros(0)] * len(plan.radices)
    for t in range(len(plan.radices) - 1, -1, -1):
        b, s = plan.radices[t], strides[t]
        grp = plan.d // (b * s)
        vt = states[t].reshape(n, grp, b, s)                   # [row][alpha][i][beta]
        gt = g.reshape(n, grp, b, s)                           # [row][alpha][j][beta]
        grads[t] = np.einsum("naib,najb->abij", vt, gt).reshape(grp * s, b, b)   # block c = alpha*s + beta
        g = _stage(g, b, s, plan.blocks[t], transposed=True)   # gradient with respect to v_t
    return grads


def forward_passes(plans: Sequence[OraclePlan], x: np.ndarray) -> np.ndarray:
    """Several passes (Section "HARP processors"): y = x . Q_0 . Q_1 ... , each Q_k one processor."""
    y = np.array(x, dtype=np.float64, ndmin=2)
    for p in plans:
        y = forward(p, y)
    return y


def transpose_passes(plans: Sequence[OraclePlan], y: np.ndarray) -> np.ndarray:
    """x = y . Q_{n-1}^T ... Q_0^T, the inverse of forward_passes for orthogonal blocks."""
    x = np.array(y, dtype=np.float64, ndmin=2)
    for p in reversed(list(plans)):
        x = transpose(p, x)
    return x


def dense(plan: OraclePlan) -> np.ndarray:
    """Materialise Q (d x d) with forward(x) == x @ Q, by pushing the identity through."""
    return forward(plan, np.eye(plan.d))


def rel_err_rows(got: np.ndarray, want: np.ndarray) -> float:
    """max over rows of max_i |got_i - want_i| / ||want||_2 (the parity metric)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    nrm = np.linalg.norm(want, axis=1)
    nrm = np.where(nrm == 0.0, 1.0, nrm)
    return float(np.max(np.max(np.abs(got - want), axis=1) / nrm)) if got.size else 0.0
