"""The multi-GPU leg of the benchmark is "replicas only": ranks share nothing but the timing
reduction.  This runs that reduction on two gloo ranks on the CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, results):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0 took 10 ms, rank 1 took 20 ms for 100 units each: the job rate is 2*100 / 20 ms
    rate, tmax, w = bench.aggregate_rate(10.0 * (rank + 1), 100, dist, None)
    results[rank] = (rate, tmax, w)
    dist.destroy_process_group()


def test_replica_rates_add_and_the_slowest_rank_sets_the_time():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        results = m.dict()
        port = 29500 + (os.getpid() % 2000)
        procs = [ctx.Process(target=_rank_main, args=(r, 2, port, results)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(timeout=120)
            assert p.exitcode == 0
        for r in range(2):
            rate, tmax, w = results[r]
            assert w == 2 and tmax == 20.0
            assert abs(rate - 2 * 100 / 0.020) < 1e-6


def test_single_process_rate():
    sys.path.insert(0, ROOT)
    import bench
    rate, tmax, w = bench.aggregate_rate(5.0, 32, None, None)
    assert w == 1 and tmax == 5.0 and abs(rate - 32 / 0.005) < 1e-9
