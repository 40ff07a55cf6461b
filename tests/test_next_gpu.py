"""Plan helpers and the symmetric two-sided product on the GPU, against the oracles."""
import numpy as np
import pytest
import scipy.linalg
import torch

import paper_2605_29843_b200 as harp
from oracle import harp_oracle as orc
from oracle import harp_params as prm
from paper_2605_29843_b200 import workloads as wl
from harp_testlib import TOL, gpu_apply, host_rows, promote, to_device, to_host_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("radices", [(2, 2, 2, 4), (8, 8), (4, 2, 8, 5), (16, 2)])
@pytest.mark.parametrize("int8", [False, True])
def test_plan_from_theta(radices, int8):
    d = int(np.prod(radices))
    rng = np.random.default_rng(17)
    theta, mixers, blocks64, tq, sc = [], [], [], [], []
    for b in radices:
        th = rng.normal(0, 0.25, (d // b, prm.n_params(b)))
        mixer = None if (b & (b - 1)) == 0 else np.linalg.qr(rng.standard_normal((b, b)))[0]
        if int8:
            q, s = prm.quantize_theta(th)
            s = s.astype(np.float32)
            tq.append(q); sc.append(s)
            th = prm.dequantize_theta(q, s.astype(np.float64))
        theta.append(th.astype(np.float32))
        mixers.append(None if mixer is None else mixer.astype(np.float32))
        blocks64.append(prm.blocks_from_theta(b, theta[-1].astype(np.float64) if not int8 else th,
                                              None if mixer is None else mixer.astype(np.float32).astype(np.float64)))
    signs = wl.rademacher(rng, d)
    perm = rng.permutation(d).astype(np.int32)
    plan = harp.harp_plan_create_from_theta(d, radices, perm, signs, theta=None if int8 else theta,
                                            theta_q=tq if int8 else None, scales=sc if int8 else None, mixers=mixers)
    oplan = orc.OraclePlan(d, radices, perm, signs, blocks64)
    xh = host_rows(rng.standard_normal((13, d)), "f32")
    got, guards = gpu_apply(plan, xh, "f32")
    assert guards and orc.rel_err_rows(got, orc.forward(oplan, promote(xh, "f32"))) <= TOL["f32"]
    got, guards = gpu_apply(plan, xh, "f32", True)
    assert guards and orc.rel_err_rows(got, orc.transpose(oplan, promote(xh, "f32"))) <= TOL["f32"]


@pytest.mark.parametrize("K,rows", [(2, None), (4, [1, 3, 0, 2]), (8, [5, 0, 7, 2, 1, 6, 3, 4])])
def test_kronecker_fallback_plan(K, rows):
    hk = scipy.linalg.hadamard(K).astype(np.float64)
    if rows is not None:
        hk = hk[rows]
    radices, n2 = (4, 2, 4), 32
    rng = np.random.default_rng(23)
    blocks = [wl.qr_orthogonal(rng, n2 // b, b).astype(np.float32) for b in radices]
    plan = harp.harp_plan_create_kronecker(n2, radices, blocks, K, hk)
    d = K * n2
    assert harp.harp_plan_dim(plan) == d
    t_small = orc.dense(orc.OraclePlan(n2, radices, None, None, blocks))
    want = np.kron(hk / np.sqrt(K), t_small)
    eye = np.eye(d, dtype=np.float32)
    got, guards = gpu_apply(plan, eye, "f32")                 # rows of I through the plan = the dense matrix
    assert guards and np.max(np.abs(got - want)) < 2e-6
    # a table that is not a Hadamard table is rejected
    bad = hk.copy()
    bad[0, 0] = -bad[0, 0]
    with pytest.raises(harp.HarpError):
        harp.harp_plan_create_kronecker(n2, radices, blocks, K, bad)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_symmetric_two_sided_product(dtype):
    """H~ = V^T H V (second moment rotated on both sides with the same processor)."""
    spec = wl.make_plan(61, 512, (8, 8, 8), "qr", perm="identity", signs=True)
    V = orc.dense(orc.OraclePlan.from_spec(spec))
    rng = np.random.default_rng(29)
    X = rng.standard_normal((700, 512)) * (1.0 + 5.0 * (rng.random(512) < 0.02))
    H = X.T @ X / 700.0
    hh = host_rows(H, dtype)
    h64 = promote(hh, dtype)
    hd = to_device(hh, dtype)
    plan = harp.plan_from_spec(spec)
    harp.two_sided_(hd, plan, plan)
    torch.cuda.synchronize()
    got = to_host_f64(hd)
    want = V.T @ h64 @ V
    scale = np.minimum(np.linalg.norm(want, axis=1, keepdims=True), np.linalg.norm(want, axis=0, keepdims=True))
    assert np.max(np.abs(got - want) / scale) <= 2 * TOL[dtype]
    assert abs(np.trace(got) - np.trace(h64)) / np.trace(h64) < (1e-5 if dtype == "f32" else 5e-3)
    assert np.max(np.abs(got - got.T) / scale) <= 4 * TOL[dtype]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_passes(dtype):
    """Two and three passes against the oracle's composition, forward and transpose."""
    specs = [wl.tiny_plan(11, (4, 4, 4, 4), kind="qr", perm="random", signs=True),
             wl.tiny_plan(12, (16, 16), kind="qr", perm="identity", signs=False),
             wl.tiny_plan(13, (2, 8, 16), kind="qr", perm="identity", signs=True)]
    plans = [harp.plan_from_spec(sp) for sp in specs]
    oplans = [orc.OraclePlan.from_spec(sp) for sp in specs]
    rng = np.random.default_rng(21)
    xh = host_rows(rng.standard_normal((33, 256)), dtype)
    x64 = promote(xh, dtype)
    code = harp.HARP_F32 if dtype == "f32" else harp.HARP_BF16
    for n in (2, 3):
        for tr in (False, True):
            x = to_device(xh, dtype)
            harp.harp_apply_passes(plans[:n], x.data_ptr(), 33, code, tr, torch.cuda.current_stream().cuda_stream)
            want = orc.transpose_passes(oplans[:n], x64) if tr else orc.forward_passes(oplans[:n], x64)
            assert orc.rel_err_rows(to_host_f64(x), want) <= n * TOL[dtype]
    with pytest.raises(harp.HarpError):
        harp.harp_apply_passes([plans[0], harp.plan_from_spec(wl.tiny_plan(1, (4, 4), kind="qr"))],
                               to_device(xh, dtype).data_ptr(), 33, code)


@pytest.mark.parametrize("n_rows", [1, 16, 64])
def test_small_batches_chained_and_in_a_cuda_graph(n_rows):
    """Wide rows, few rows (the decode case): consecutive applies on a side stream overlap each
    kernel's preamble with the kernel before it.  A forward/transpose chain must give the same bits
    whether launched call by call or replayed from a CUDA graph, and match the oracle."""
    w = wl.config(4)
    spec = w.plans["q"]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(90 + n_rows)
    xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
    side = torch.cuda.Stream()

    def chain(x, st):
        for k in range(5):                                  # F T F T F: one forward in total
            harp.harp_apply(plan, x.data_ptr(), n_rows, harp.HARP_BF16, bool(k & 1), st)

    eager = to_device(xh, "bf16")
    with torch.cuda.stream(side):
        chain(eager, side.cuda_stream)
    side.synchronize()
    replayed = to_device(xh, "bf16")
    graph = torch.cuda.CUDAGraph()
    scratch = to_device(xh, "bf16")
    with torch.cuda.stream(side):
        chain(scratch, side.cuda_stream)                    # warm-up before capture
        side.synchronize()
        scratch.copy_(replayed)
        with torch.cuda.graph(graph, stream=side):
            chain(scratch, side.cuda_stream)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(eager.view(torch.int16), scratch.view(torch.int16))
    # five roundings to bf16 along the chain: a few times the single-apply tolerance
    want = orc.forward(oplan, promote(xh, "bf16"))
    assert orc.rel_err_rows(to_host_f64(eager), want) <= 3 * TOL["bf16"]


@pytest.mark.parametrize("cfg,n_rows", [(2, 48), (2, 16 * 300 + 5), (4, 2048)])
def test_dependent_launches_chained_and_in_a_cuda_graph(cfg, n_rows):
    """The whole-row kernel (cfg2) and the tensor-memory slab pass (cfg4 from 1024 rows on) start their
    preamble while the kernel before them in the stream is still running and touch the rows only after it has
    completed.  A forward/transpose chain on a side stream must give the same bits whether launched call by
    call or replayed from a CUDA graph, and match the oracle on a sample of rows."""
    spec = wl.config(cfg).plans["q"]
    plan = harp.plan_from_spec(spec)
    oplan = orc.OraclePlan.from_spec(spec)
    rng = np.random.default_rng(190 + n_rows)
    xh = host_rows(rng.standard_normal((n_rows, spec.d)), "bf16")
    side = torch.cuda.Stream()

    def chain(x, st):
        for k in range(5):                                  # F T F T F: one forward in total
            harp.harp_apply(plan, x.data_ptr(), n_rows, harp.HARP_BF16, bool(k & 1), st)

    eager = to_device(xh, "bf16")
    with torch.cuda.stream(side):
        chain(eager, side.cuda_stream)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    scratch = to_device(xh, "bf16")
    fresh = to_device(xh, "bf16")
    with torch.cuda.stream(side):
        chain(scratch, side.cuda_stream)                    # warm-up before capture
        side.synchronize()
        scratch.copy_(fresh)
        with torch.cuda.graph(graph, stream=side):
            chain(scratch, side.cuda_stream)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(eager.view(torch.int16), scratch.view(torch.int16))
    pick = np.unique(np.concatenate([np.arange(min(n_rows, 24)), np.arange(max(0, n_rows - 24), n_rows)]))
    want = orc.forward(oplan, promote(xh[pick], "bf16"))
    assert orc.rel_err_rows(to_host_f64(eager)[pick], want) <= 3 * TOL["bf16"]
    assert harp.harp_plan_error_word(plan) == 0
