"""The plain-C oracle must agree with the numpy oracle (itself pinned in
test_oracle_pins.py) and with a dense product."""
import numpy as np
import pytest

from oracle import c_oracle, harp_oracle as orc
from paper_2605_29843_b200 import workloads as wl


@pytest.mark.parametrize("radices", [(2, 2, 2), (7, 2), (3, 5, 2), (16, 4), (43,), (4, 3, 8, 5)])
@pytest.mark.parametrize("perm", ["identity", "random"])
def test_c_matches_numpy(radices, perm):
    spec = wl.tiny_plan(13, radices, kind="qr", perm=perm, signs=True)
    plan, cplan = orc.OraclePlan.from_spec(spec), c_oracle.CPlan(spec)
    x = np.random.default_rng(2).standard_normal((9, spec.d))
    assert np.allclose(c_oracle.forward(cplan, x), orc.forward(plan, x), atol=1e-13, rtol=0)
    assert np.allclose(c_oracle.transpose(cplan, x), orc.transpose(plan, x), atol=1e-13, rtol=0)
    Q = orc.dense(plan)
    assert np.allclose(c_oracle.forward(cplan, x), x @ Q, atol=1e-12, rtol=0)


def test_c_matches_numpy_config_sizes():
    for cfg in (2, 3):
        w = wl.config(cfg, n_rows=3)
        spec = w.plans["q"]
        x = w.data["x"].rows_f64(0, 3)
        a = c_oracle.forward(c_oracle.CPlan(spec), x)
        b = orc.forward(orc.OraclePlan.from_spec(spec), x)
        assert orc.rel_err_rows(a, b) < 1e-14


def test_c_two_sided_matches_numpy():
    p_out = wl.tiny_plan(21, (3, 4))
    p_in = wl.tiny_plan(22, (2, 5, 2))
    W = np.random.default_rng(3).standard_normal((12, 20))
    a = c_oracle.two_sided(c_oracle.CPlan(p_out), c_oracle.CPlan(p_in), W)
    b = orc.two_sided(orc.OraclePlan.from_spec(p_out), orc.OraclePlan.from_spec(p_in), W)
    assert np.allclose(a, b, atol=1e-13, rtol=0)


def test_threads_reported():
    assert c_oracle.threads() >= 1
