"""The layer-sharded form on several ranks, on the CPU: every rank (a gloo process standing for a
GPU) runs the oracle's pass of its own shard -- rank = shard, world size = shard count, the mapping
a multi-GPU launch uses -- and the ranks then compare notes: every layer has exactly one owner,
and the owners' gradients put together are the sequential pass.  Nothing is exchanged before that.
The rank -> shard mapping is the product's own (`bench.shard_plan`, what `bench.py --gpus N
--shard-by-rank` runs), and the layers a rank claims come from the library's rule -- layer l
belongs to shard (L - l) mod S, worker ((L - l) / S) mod k inside it -- checked against what the
oracle's shard pass really wrote."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, results):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import lf_inputs
    from oracle import lf_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    L, N, B, k = 5, 12, 2, 4
    S, r, k_here = bench.shard_plan(world, rank, k, 1, True)     # the product's mapping of ranks to shards
    assert (S, r) == (world, rank) and k_here == max(1, k // world)
    assert bench.shard_plan(1, 0, k, 1, True) == (1, 0, k)       # one rank: no sharding
    assert bench.shard_plan(1, 0, k, 4, False) == (4, 0, 1)      # --shards 4 on one GPU: shard 0, k / 4 workers
    mine = [l for l in range(1, L + 1) if (L - l) % S == r]      # the library's ownership rule
    workers = sorted({((L - l) // S) % k_here for l in mine})
    assert workers == list(range(min(k_here, len(mine))))        # the shard's layers go round its workers
    t = lf_inputs.make_inputs(L, N, B, "uniform", lf_inputs.SEED_BASE + 31, "cpu")   # same seed: replicated inputs
    w = t["w"].numpy()
    z, a = orc.forward(w, t["b"].numpy(), t["x"].numpy())
    delta, gw, gb, wrote = orc.backward_shard(w, z, a, t["y"].numpy(), S, r)
    assert [l for l in range(1, L + 1) if wrote[l - 1]] == mine  # the oracle's shard wrote exactly those
    owners = torch.from_numpy(wrote.astype(np.int64))
    dist.all_reduce(owners)                                   # how many ranks own each layer
    parts = torch.from_numpy(np.nan_to_num(gw, nan=0.0))
    dist.all_reduce(parts)                                    # the owners' gradients put together
    d_all = [torch.zeros_like(torch.from_numpy(delta)) for _ in range(world)]
    dist.all_gather(d_all, torch.from_numpy(delta))           # every rank's copy of the chain
    _, gw_seq, _ = orc.backward_sequential(w, z, a, t["y"].numpy())
    results[rank] = (owners.tolist(), bool(np.array_equal(parts.numpy(), gw_seq)),
                     all(bool(torch.equal(d, d_all[0])) for d in d_all))
    dist.destroy_process_group()


def test_two_ranks_own_disjoint_layers_and_together_give_the_full_gradient():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        results = m.dict()
        port = 31500 + (os.getpid() % 2000)
        procs = [ctx.Process(target=_rank_main, args=(r, 2, port, results)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(timeout=180)
            assert p.exitcode == 0
        for r in range(2):
            owners, same_gw, same_delta = results[r]
            assert owners == [1] * 5 and same_gw and same_delta
