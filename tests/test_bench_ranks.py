"""The multi-process part of bench.py on CPU: world size 2 over gloo.

The sweep does not shard (one GPU, no collectives on the data path): `bench.py --gpus N` runs N
independent replicas, and the only cross-rank step is how their timings and token counts are
combined -- the slowest rank's time, the sum of the tokens.  That step is checked here.
"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, tokens = bench.over_ranks(dist, "cpu", 10.0 + 5.0 * rank, 1000 * (rank + 1))
    dist.barrier()
    out[rank] = (ms, tokens)
    dist.destroy_process_group()


def test_replica_timings_combine_as_max_and_sum():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1] == (15.0, 3000.0)


def test_single_process_is_identity():
    import bench
    assert bench.over_ranks(None, "cpu", 7.5, 123) == (7.5, 123.0)
