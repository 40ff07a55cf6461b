"""Row sharding over ranks (world_size 2, gloo, CPU): the apply path has no data-path
collective, so N ranks that each transform their own row range must reproduce the
single-process result exactly; the only collective is the max-over-ranks of the timing."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


from paper_2605_29843_b200 import shard_rows  # noqa: E402


def _worker(rank, world, port, n_rows, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import harp_oracle as orc
    from paper_2605_29843_b200 import workloads as wl
    spec = wl.tiny_plan(5, (4, 3, 2, 5), perm="random")
    plan = orc.OraclePlan.from_spec(spec)
    data = wl.DataSpec(n_rows, spec.d, "f32", "normal", seed=9)
    a, b = shard_rows(n_rows, rank, world)
    y = orc.forward(plan, data.rows_f64(a, b - a)) if b > a else np.zeros((0, spec.d))
    np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
    # the benchmark's timing reduction: max over ranks
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == float(world)
    dist.barrier()
    dist.destroy_process_group()


def test_shard_rows_partition():
    for n in (0, 1, 7, 16, 1001):
        for world in (1, 2, 3, 8):
            spans = [shard_rows(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            assert max(b - a for a, b in spans) - min(b - a for a, b in spans) <= 1


def test_two_ranks_reproduce_single_process(tmp_path):
    from oracle import harp_oracle as orc
    from paper_2605_29843_b200 import workloads as wl
    n_rows, world = 37, 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(world, port, n_rows, str(tmp_path)), nprocs=world, join=True)
    spec = wl.tiny_plan(5, (4, 3, 2, 5), perm="random")
    whole = orc.forward(orc.OraclePlan.from_spec(spec), wl.DataSpec(n_rows, spec.d, "f32", "normal", seed=9).rows_f64(0, n_rows))
    parts = np.concatenate([np.load(tmp_path / f"y{r}.npy") for r in range(world)])
    assert np.array_equal(parts, whole)
