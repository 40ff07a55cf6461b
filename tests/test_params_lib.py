"""Host-side plan helpers of the library against the plan-side oracle (no GPU needed)."""
import os

import numpy as np
import pytest

import paper_2605_29843_b200 as harp
from oracle import harp_params as prm
from paper_2605_29843_b200 import build as harp_build

GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module", autouse=True)
def _built():
    harp_build.build()


def test_greedy_schedule_golden_and_oracle():
    for line in open(os.path.join(GOLD, "greedy_schedule.txt")):
        if line.startswith("#") or not line.strip():
            continue
        d, bb, bm, sched = line.split()
        assert harp.harp_greedy_schedule(int(d), int(bb), int(bm)) == [int(v) for v in sched.split(",")]
    for d in (2, 3, 60, 97, 11008, 12288, 14336, 22016, 28672, 65536, 1 << 20):
        for bb, bm in ((8, 8), (16, 16), (4, 8), (2, 16)):
            assert harp.harp_greedy_schedule(d, bb, bm) == prm.greedy_schedule(d, bb, bm)
    assert harp.lib().harp_greedy_schedule(1, 8, 8, None, 4) == -1


@pytest.mark.parametrize("b", [2, 3, 4, 5, 7, 8, 16, 43])
def test_blocks_from_theta_match_oracle(b):
    rng = np.random.default_rng(b)
    npar = harp.harp_theta_params_per_block(b)
    assert npar == prm.n_params(b)
    theta = rng.normal(0, 0.3, (9, npar)).astype(np.float32)
    mixer = None if (b & (b - 1)) == 0 else np.linalg.qr(rng.standard_normal((b, b)))[0].astype(np.float32)
    got = harp.harp_blocks_from_theta(b, theta=theta, mixer=mixer)
    want = prm.blocks_from_theta(b, theta.astype(np.float64), None if mixer is None else mixer.astype(np.float64))
    assert np.max(np.abs(got - want)) < 2e-7
    # theta = 0 returns the mixer itself; blocks are orthogonal
    zero = harp.harp_blocks_from_theta(b, theta=np.zeros((1, npar), np.float32), mixer=mixer)
    g = prm.sylvester(b) if mixer is None else mixer
    assert np.max(np.abs(zero[0] - g)) < 1e-7
    assert np.max(np.abs(np.swapaxes(got, 1, 2).astype(np.float64) @ got - np.eye(b))) < 2e-6


@pytest.mark.parametrize("b", [2, 3, 4, 5, 7, 8, 16, 43])
def test_grad_theta_matches_oracle(b):
    rng = np.random.default_rng(60 + b)
    npar = harp.harp_theta_params_per_block(b)
    theta = rng.normal(0, 0.3, (7, npar)).astype(np.float32)
    gb = rng.standard_normal((7, b, b)).astype(np.float32)
    mixer = None if (b & (b - 1)) == 0 else np.linalg.qr(rng.standard_normal((b, b)))[0].astype(np.float32)
    got = harp.harp_grad_theta(b, theta, gb, mixer)
    want = prm.grad_theta(b, theta.astype(np.float64), gb.astype(np.float64), None if mixer is None else mixer.astype(np.float64))
    assert got.shape == want.shape == (7, npar)
    assert np.max(np.abs(got - want)) <= 1e-6 * max(1.0, np.max(np.abs(want)))
    L = harp.lib()
    assert L.harp_grad_theta(b, 7, None, None, gb.ctypes.data, got.ctypes.data) == 1
    assert L.harp_grad_theta(1, 7, theta.ctypes.data, None, gb.ctypes.data, got.ctypes.data) == 3
    if mixer is not None:                                     # no default mixer for this radix
        assert L.harp_grad_theta(b, 7, theta.ctypes.data, None, gb.ctypes.data, got.ctypes.data) == 1


def test_int8_parameters():
    rng = np.random.default_rng(5)
    b = 8
    theta = rng.normal(0, 0.2, (6, 28))
    q, s = prm.quantize_theta(theta)
    got = harp.harp_blocks_from_theta(b, theta_q=q, scales=s)
    want = prm.blocks_from_theta(b, prm.dequantize_theta(q, s.astype(np.float32).astype(np.float64)))
    assert np.max(np.abs(got - want)) < 2e-7


def test_missing_mixer_is_an_error():
    st = harp.lib().harp_blocks_from_theta(3, 1, np.zeros(3, np.float32).ctypes.data, None, None, None,
                                           np.zeros(9, np.float32).ctypes.data)
    assert st == 1
