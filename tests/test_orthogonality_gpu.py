"""What the bf16 tensor-core paths do to a row as an orthogonal map: block kernels rounded to bf16 and
rows rounded to bf16 after every fused phase (2 to 5 roundings per coordinate).  Bounds on the
forward-then-transpose round trip and on the drift of the row norm, on the configurations' own data
(heavy tails, outlier channels x100), with the kernels HARP_KERNEL_AUTO picks."""
import numpy as np
import pytest
import torch

import paper_2605_29843_b200 as harp
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import TOL, promote, to_device, to_host_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,n_rows", [(2, 2048), (3, 1536), (4, 1536), (5, 512)])
def test_round_trip_and_norm_drift(cfg, n_rows):
    w = wl.config(cfg)
    spec = w.plans["in"] if cfg == 5 else w.plans["q"]
    data = w.data["x"]
    plan = harp.plan_from_spec(spec)
    xh = data.rows(0, n_rows)
    x64 = promote(xh, "bf16")
    x = to_device(xh, "bf16")
    harp.apply_(plan, x)
    torch.cuda.synchronize()
    y = to_host_f64(x)
    nx, ny = np.linalg.norm(x64, axis=1), np.linalg.norm(y, axis=1)
    # Q is orthogonal: the norm of every row survives, up to the roundings.  One rounding moves a
    # coordinate by at most 2^-9 of its size, hence the norm by at most 2^-9 (reached when one coordinate
    # carries the row, as in the heavy-tailed rows); at most four roundings per coordinate on these plans
    drift = float(np.max(np.abs(ny / nx - 1.0)))
    assert drift <= 4 * 2.0 ** -9, drift
    harp.apply_(plan, x, transpose=True)
    torch.cuda.synchronize()
    back = to_host_f64(x)
    # forward then transpose is the identity: two applies' worth of error, relative to the row norm
    err = float(np.max(np.max(np.abs(back - x64), axis=1) / nx))
    assert err <= 2 * TOL["bf16"], err
    # and the error does not pile up on the outlier channels' rows more than elsewhere: same bound per row
    assert harp.harp_plan_error_word(plan) == 0
