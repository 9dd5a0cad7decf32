"""The N > 1 path of the benchmark is replicas only: the only cross-rank logic is the max-over-ranks of
the device times and the aggregate throughput.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times = [(1.0, 0.40, 4.0), (1.5, 0.50, 3.0)][rank]
    out = bench.aggregate_over_ranks(dist, torch.device("cpu"), world, 2.0e12, *times)
    dist.barrier()
    q.put((rank, out))
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_max_time_and_sums_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank in (0, 1):
        ms, head, e2e, value, e2e_value = res[rank]
        assert (ms, head, e2e) == (1.5, 0.50, 4.0)
        assert abs(value - 2 * 2.0e12 / 0.5e-3 / 1e12) < 1e-9
        assert abs(e2e_value - 2 * 2.0e12 / 4.0e-3 / 1e12) < 1e-9


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    ms, head, e2e, value, e2e_value = bench.aggregate_over_ranks(None, torch.device("cpu"), 1, 1.0e12, 2.0, 0.5, 5.0)
    assert (ms, head, e2e) == (2.0, 0.5, 5.0) and abs(value - 2000.0) < 1e-9 and abs(e2e_value - 200.0) < 1e-9
