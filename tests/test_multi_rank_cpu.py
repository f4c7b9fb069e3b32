"""The N > 1 path of the benchmark has no data-path collective (replicas only); what it does across
ranks -- distinct seeds per rank, time = max over ranks, work = sum over ranks -- is checked here with
two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                    # rank 1 is the slow one
    ms, seqs, value = bench.aggregate(ms_local, 3072 * (rank + 1), dist, "cpu")
    out.put((rank, ms, seqs, value, bench.rank_seed(rank)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_max_time_and_sums_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, seqs, value, seed in res:
        assert ms == 15.0 and seqs == 3072 * 3 and abs(value - 9216 / 0.015) < 1e-6
    assert res[0][4] != res[1][4]                  # replicas draw different data


def test_single_rank_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(2.0, 100) == (2.0, 100.0, 50000.0)
