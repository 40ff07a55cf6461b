"""Seeded synthetic inputs for the HARP apply path.

This module only *draws inputs*: processor parameters (schedule, Rademacher
signs, fixed permutation, orthogonal block kernels) and data rows with the tail
structure of LLM activations and weights.  It applies no processor to any
data -- neither the CPU oracle nor the CUDA library is imported here, and both
consume exactly the arrays produced here (blocks already rounded to fp32, data
already rounded to the I/O dtype).

Block kernels follow the paper's block form B = Q(theta) G_b (Eq. 9): a
normalised Sylvester Hadamard mixer for power-of-two radices and a QR-of-
Gaussian orthogonal mixer otherwise; Q(theta) is a Givens rotation for b = 2
(Eq. 10).  Everything is numpy; randomness comes from numpy's PCG64
``default_rng`` with explicit integer seeds.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------
# dtype helpers (bf16 is carried as uint16 bit patterns on the host)
# --------------------------------------------------------------------------


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact promotion of bf16 bit patterns to fp64."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


# --------------------------------------------------------------------------
# processor description shared by both sides (pure data)
# --------------------------------------------------------------------------


@dataclass
class PlanSpec:
    """Host description of one HARP processor Q = D_s . Pi . T.

    radices : stage radices b_0..b_{m-1}, product d (Eq. 6)
    perm    : int32[d], forward gathers v[i] = u[perm[i]]; None = identity
    signs   : int8[d] in {+1,-1}; None = all +1
    blocks  : per stage t a float32 array [d/b_t, b_t, b_t]; block c = alpha*s_t+beta
              is used as out[j] = sum_i in[i] * K[c][i][j]
    """

    d: int
    radices: Tuple[int, ...]
    perm: Optional[np.ndarray]
    signs: Optional[np.ndarray]
    blocks: List[np.ndarray]
    name: str = ""

    @property
    def strides(self) -> Tuple[int, ...]:
        s, out = 1, []
        for b in self.radices:
            out.append(s)
            s *= b
        return tuple(out)


def sylvester_hadamard(b: int) -> np.ndarray:
    """Normalised Sylvester Hadamard H_b for b a power of two (fp64)."""
    assert b >= 1 and (b & (b - 1)) == 0
    h = np.ones((1, 1))
    while h.shape[0] < b:
        h = np.block([[h, h], [h, -h]])
    return h / np.sqrt(b)


def qr_orthogonal(rng: np.random.Generator, n_blocks: int, b: int) -> np.ndarray:
    """n_blocks orthogonal b x b matrices: QR of a Gaussian with diag(R) made positive."""
    g = rng.standard_normal((n_blocks, b, b))
    q, r = np.linalg.qr(g)
    sgn = np.sign(np.diagonal(r, axis1=1, axis2=2))
    sgn[sgn == 0] = 1.0
    return q * sgn[:, None, :]


def givens_times_h2(theta: np.ndarray) -> np.ndarray:
    """B = Q(theta) H_2 with Q the Givens rotation [[c,-s],[s,c]]."""
    c, s = np.cos(theta), np.sin(theta)
    q = np.stack([np.stack([c, -s], -1), np.stack([s, c], -1)], -2)
    return q @ sylvester_hadamard(2)


def expm_skew(a: np.ndarray) -> np.ndarray:
    """exp((A - A^T)/2) for a batch of small matrices via the eigen-decomposition
    of the Hermitian matrix i*S (S skew-symmetric)."""
    s = 0.5 * (a - np.swapaxes(a, -1, -2))
    w, v = np.linalg.eigh(1j * s)           # i*S is Hermitian; S = -i V diag(w) V^H
    e = (v * np.exp(-1j * w)[..., None, :]) @ np.conj(np.swapaxes(v, -1, -2))
    return np.real(e)


def digit_reversal_perm(radices: Sequence[int]) -> np.ndarray:
    """Mixed-radix digit reversal: i = sum_l i_l prod_{k<l} b_k  ->
    perm[i] = sum_l i_l prod_{k>l} b_k."""
    d = int(np.prod(radices))
    idx = np.arange(d)
    digits = []
    rem = idx.copy()
    for b in radices:
        digits.append(rem % b)
        rem //= b
    out = np.zeros(d, dtype=np.int64)
    w = 1
    for l in range(len(radices) - 1, -1, -1):
        out += digits[l] * w
        w *= radices[l]
    return out.astype(np.int32)


def rademacher(rng: np.random.Generator, d: int) -> np.ndarray:
    return (1 - 2 * rng.integers(0, 2, size=d)).astype(np.int8)


def make_blocks(rng: np.random.Generator, d: int, radices: Sequence[int], kind: str,
                sigma: float = 0.1) -> List[np.ndarray]:
    """Draw one block array per stage, rounded once to fp32.

    kind = 'givens_h2'  : radix 2 -> Q(theta) H_2, theta ~ U[-pi, pi); other radices -> QR
           'expm_h'     : pow-2 radix -> exp(skew A) H_b, A_ij ~ N(0, sigma^2); else QR
           'qr'         : QR of Gaussian, sign-fixed
           'hadamard'   : pow-2 radix -> H_b exactly (Theta = 0); else QR
           'identity'   : identity blocks (index-map tests)
    """
    out = []
    for b in radices:
        n = d // b
        pow2 = (b & (b - 1)) == 0
        if kind == "identity":
            k = np.broadcast_to(np.eye(b), (n, b, b)).copy()
        elif kind == "givens_h2" and b == 2:
            k = givens_times_h2(rng.uniform(-np.pi, np.pi, size=n))
        elif kind == "expm_h" and pow2:
            a = rng.normal(0.0, sigma, size=(n, b, b))
            k = expm_skew(a) @ sylvester_hadamard(b)
        elif kind == "hadamard" and pow2:
            k = np.broadcast_to(sylvester_hadamard(b), (n, b, b)).copy()
        else:
            k = qr_orthogonal(rng, n, b)
        out.append(np.ascontiguousarray(k, dtype=np.float32))
    return out


def make_plan(seed: int, d: int, radices: Sequence[int], kind: str, perm: str = "identity",
              signs: bool = True, sigma: float = 0.1, name: str = "") -> PlanSpec:
    """Draw order: signs, perm, blocks of stage 0, 1, ..."""
    assert int(np.prod(radices)) == d
    rng = np.random.default_rng(seed)
    sg = rademacher(rng, d) if signs else None
    if perm == "identity":
        pm = None
    elif perm == "digit_reversal":
        pm = digit_reversal_perm(radices)
    elif perm == "random":
        pm = rng.permutation(d).astype(np.int32)
    else:
        raise ValueError(perm)
    blocks = make_blocks(rng, d, radices, kind, sigma)
    return PlanSpec(d, tuple(int(b) for b in radices), pm, sg, blocks, name)


# --------------------------------------------------------------------------
# data rows, drawn in fixed-size chunks so any row range can be regenerated
# --------------------------------------------------------------------------

ROW_CHUNK = 256


@dataclass
class DataSpec:
    n_rows: int
    d: int
    dtype: str                    # 'f32' | 'bf16'
    dist: str                     # 'normal' | 'student_t3'
    scale: float = 1.0
    outlier_frac: float = 0.0     # ceil(frac*d) channels, fixed per config
    outlier_gain: float = 1.0
    seed: int = 0

    def outlier_channels(self) -> np.ndarray:
        n = int(np.ceil(self.outlier_frac * self.d)) if self.outlier_frac > 0 else 0
        if n == 0:
            return np.zeros(0, dtype=np.int64)
        rng = np.random.default_rng([self.seed, 0x0C4A])
        return np.sort(rng.choice(self.d, size=n, replace=False))

    def _chunk(self, k: int) -> np.ndarray:
        rng = np.random.default_rng([self.seed, 0xDA7A, k])
        shape = (ROW_CHUNK, self.d)
        if self.dist == "normal":
            x = rng.standard_normal(shape, dtype=np.float32)
        elif self.dist == "student_t3":
            x = rng.standard_t(3.0, size=shape).astype(np.float32)
        else:
            raise ValueError(self.dist)
        if self.scale != 1.0:
            x *= np.float32(self.scale)
        ch = self.outlier_channels()
        if ch.size:
            x[:, ch] *= np.float32(self.outlier_gain)
        return x

    def rows(self, start: int, count: int) -> np.ndarray:
        """Rows [start, start+count) in the I/O dtype: float32 array for 'f32',
        uint16 bf16 bit patterns for 'bf16'."""
        assert 0 <= start and start + count <= self.n_rows
        out = np.empty((count, self.d), dtype=np.float32)
        r = start
        while r < start + count:
            k, off = divmod(r, ROW_CHUNK)
            take = min(ROW_CHUNK - off, start + count - r)
            out[r - start:r - start + take] = self._chunk(k)[off:off + take]
            r += take
        return out if self.dtype == "f32" else f32_to_bf16_bits(out)

    def rows_f64(self, start: int, count: int) -> np.ndarray:
        """The same rows, promoted exactly to fp64 (what the oracle consumes)."""
        r = self.rows(start, count)
        return r.astype(np.float64) if self.dtype == "f32" else bf16_bits_to_f64(r)


# --------------------------------------------------------------------------
# the five benchmark configurations
# --------------------------------------------------------------------------


@dataclass
class Workload:
    name: str
    plans: Dict[str, PlanSpec]
    data: Dict[str, DataSpec]
    tol: float
    notes: str = ""
    extra: dict = field(default_factory=dict)


def config(idx: int, n_rows: Optional[int] = None) -> Workload:
    """Configuration idx in 1..5; n_rows overrides the activation row count
    (the plan and the per-chunk data do not depend on it)."""
    if idx == 1:
        d, rad = 2048, (2,) * 11
        plan = make_plan(0, d, rad, "givens_h2", name="cfg1")
        data = DataSpec(n_rows or 4096, d, "f32", "normal", outlier_frac=0.01,
                        outlier_gain=50.0, seed=100)
        return Workload("cfg1_d2048_radix2_f32", {"q": plan}, {"x": data}, 1e-5)
    if idx == 2:
        d, rad = 4096, (4,) * 6
        plan = make_plan(1, d, rad, "expm_h", perm="digit_reversal", sigma=0.1, name="cfg2")
        data = DataSpec(n_rows or 16384, d, "bf16", "normal", seed=101)
        return Workload("cfg2_d4096_radix4_bf16", {"q": plan}, {"x": data}, 8e-3)
    if idx == 3:
        d, rad = 11008, (2,) * 8 + (43,)
        plan = make_plan(2, d, rad, "givens_h2", name="cfg3")
        data = DataSpec(n_rows or 8192, d, "bf16", "student_t3", seed=102)
        return Workload("cfg3_d11008_radix2x8_43_bf16", {"q": plan}, {"x": data}, 8e-3)
    if idx == 4:
        d, rad = 14336, (16, 16, 8, 7)
        plan = make_plan(3, d, rad, "qr", name="cfg4")
        data = DataSpec(n_rows or 32768, d, "bf16", "normal", outlier_frac=0.005,
                        outlier_gain=100.0, seed=103)
        return Workload("cfg4_d14336_16_16_8_7_bf16", {"q": plan}, {"x": data}, 8e-3,
                        extra={"decode_rows": (1, 2, 4, 8, 16)})
    if idx == 5:
        p_out = make_plan(4, 8192, (8, 8, 8, 8, 2), "qr", name="cfg5_out")
        p_in = make_plan(5, 28672, (8, 8, 8, 8, 7), "qr", name="cfg5_in")
        w = DataSpec(8192, 28672, "bf16", "normal", scale=0.02, seed=104)
        x = DataSpec(n_rows or 65536, 28672, "bf16", "normal", seed=105)
        return Workload("cfg5_two_sided_8192x28672_bf16", {"out": p_out, "in": p_in},
                        {"w": w, "x": x}, 8e-3)
    raise ValueError(idx)


def tiny_plan(seed: int, radices: Sequence[int], kind: str = "qr", perm: str = "random",
              signs: bool = True) -> PlanSpec:
    d = int(np.prod(radices))
    return make_plan(seed, d, radices, kind, perm=perm, signs=signs, name="tiny")
