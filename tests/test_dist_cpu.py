"""The N > 1 bookkeeping of bench.py on CPU: two gloo ranks, no data-path collective, the
time is the max over ranks and the value is the whole job's."""
import os
import sys
from pathlib import Path

import pytest

torch = pytest.importorskip("torch")
ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, str(ROOT))
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    plan = bench.shard_plan(world, rank, 20)
    my_ms = [1.0, 3.0][rank]                        # rank 1 is the slow one
    ms, e2e = bench.reduce_max_over_ranks(torch, dist, [my_ms, 10.0 * my_ms], "cpu")
    q.put((rank, plan, ms, e2e, bench.whole_job_value(world, plan["n"], ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_bookkeeping():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, plan, ms, e2e, value in res:
        assert plan == {"rank": rank, "world": 2, "n": 1 << 20, "collectives_on_data_path": 0}
        assert ms == 3.0 and e2e == 30.0                       # max over ranks, on both ranks
        assert value == pytest.approx(2 * (1 << 20) / 3.0 / 1e6)


def test_single_process_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.reduce_max_over_ranks(torch, None, [1.5, 2.5], "cpu") == [1.5, 2.5]
    assert bench.whole_job_value(1, 1 << 30, 1.0) == pytest.approx((1 << 30) / 1e6)
