"""The N > 1 path of bench.py on CPU, two gloo ranks.

One vector is cut into contiguous shards; every rank scans its shard by itself, the 16-byte shard records
are exchanged with ONE all-gather, and every rank folds the records in front of it into its carry, which it
adds in front of its shard's first start.  Here the per-shard scans are the oracle's (with its streaming
state: a later shard honours its flag byte 0 and otherwise continues), the exchange is gloo's all-gather and
the fold is bench.fold_records; the result must equal the oracle's scan of the whole vector.  The time
bookkeeping (max over ranks, whole-job value) is checked on the way.
"""
import os
import sys
from pathlib import Path

import numpy as np
import pytest

torch = pytest.importorskip("torch")
ROOT = Path(__file__).resolve().parent.parent
LOG2N = 24                      # one generator chunk per shard


def _worker(rank, world, port, case, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, str(ROOT))
    import torch.distributed as dist
    import bench
    import mmv_inputs as gen
    import oracle
    dist.init_process_group("gloo", rank=rank, world_size=world)
    plan = bench.shard_plan(world, rank, LOG2N)
    n = plan["n"]
    x = gen.config5_values(n, first_chunk=plan["first_chunk"])
    f = gen.config5_flags(n, case, first_chunk=plan["first_chunk"])
    # the shard by itself: rank 0 starts a segment at element 0, later shards continue with a carry of zero
    state = oracle.new_f16_state()
    if rank > 0:
        state["open"] = True
    z, a = oracle.seg_scan_f16(x, f, state)
    fl = f.copy()
    if rank == 0:
        fl[0] = 1
    nz = np.flatnonzero(fl)
    first = int(nz[0]) if nz.size else n
    last_bits = int(np.array([z[-1]], dtype=np.float32).view(np.uint32)[0])
    mine = torch.from_numpy(bench.shard_record(last_bits, first, n))
    gathered = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(gathered, mine)                              # the one exchange
    records = torch.stack(gathered).numpy()
    carry = bench.fold_records(records, rank)
    z[:first] += float(carry)
    # the whole vector, scanned by the oracle in one go
    xw = gen.config5_values(world * n)
    fw = gen.config5_flags(world * n, case)
    zw, aw = oracle.seg_scan_f16(xw, fw)
    ok, ratio, i = oracle.check_fp(z.astype(np.float32), zw[rank * n:(rank + 1) * n], aw[rank * n:(rank + 1) * n])
    same_inputs = bool(np.array_equal(x, xw[rank * n:(rank + 1) * n]) and np.array_equal(f, fw[rank * n:(rank + 1) * n]))
    my_ms = [1.0, 3.0][rank]                        # rank 1 is the slow one
    ms, e2e = bench.reduce_max_over_ranks(torch, dist, [my_ms, 10.0 * my_ms], "cpu")
    q.put((rank, plan, ok, float(ratio), same_inputs, first, ms, e2e, bench.whole_job_value(world, plan["n"], ms)))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("case", ["p1e-6", "p1e-3"])
def test_two_shards_one_exchange_match_the_whole_vector(case):
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000) + (7 if case == "p1e-3" else 0)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, case, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    n = 1 << LOG2N
    for rank, plan, ok, ratio, same_inputs, first, ms, e2e, value in res:
        assert plan == {"rank": rank, "world": 2, "n": n, "global_n": 2 * n, "first_chunk": rank,
                        "collectives_on_data_path": 1}
        assert same_inputs, "a shard must hold the whole vector's values at its place"
        assert ok, f"rank {rank}: |err|/bound = {ratio}"
        assert ms == 3.0 and e2e == 30.0                       # max over ranks, on both ranks
        assert value == pytest.approx(2 * n / 3.0 / 1e6)
    if case == "p1e-6":
        assert res[1][5] > 1000       # the second shard really continues a segment of the first for a while


def test_fold_of_shard_records_is_the_segmented_operator():
    sys.path.insert(0, str(ROOT))
    import bench

    def bits(v):
        return int(np.array([v], dtype=np.float32).view(np.uint32)[0])
    n = 100
    recs = np.stack([bench.shard_record(bits(1.5), 0, n),        # has a start, ends with 1.5 open
                     bench.shard_record(bits(2.0), n, n),        # no start: continues
                     bench.shard_record(bits(-4.0), 7, n),       # start at 7: cuts the chain
                     bench.shard_record(bits(0.25), n, n)])
    assert [float(bench.fold_records(recs, r)) for r in range(5)] == [0.0, 1.5, 3.5, -4.0, -3.75]
    # integers wrap modulo 2^32
    ri = np.stack([bench.shard_record(0x7fffffff, 0, n), bench.shard_record(1, n, n)])
    assert bench.fold_records(ri, 2, is_float=False) == -(1 << 31)


def test_single_process_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.reduce_max_over_ranks(torch, None, [1.5, 2.5], "cpu") == [1.5, 2.5]
    assert bench.whole_job_value(1, 1 << 30, 1.0) == pytest.approx((1 << 30) / 1e6)
    assert bench.shard_plan(1, 0, 20)["collectives_on_data_path"] == 0
