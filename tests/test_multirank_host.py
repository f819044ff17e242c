"""Host-side logic of the N > 1 path, on CPU with gloo (world size 2): replicas draw independent
trajectories, timings reduce with max, unit counts with sum.  The data path has no collective."""
import os
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from paper_2512_22560_b200 import workloads as W
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    layout = W.make_layout(W.CONFIGS[1], seed=bench.rank_seed(W.MASTER_SEED, rank))
    local_ms = [10.0 + rank, 5.0 - rank, 1.0]
    maxima, sums = bench.reduce_over_ranks(dist, torch.device("cpu"), local_ms, [layout.spec.num_traj, int(layout.seq_lens_before.sum())])
    dist.barrier()
    q.put((rank, maxima, sums, int(layout.seq_lens_before.sum())))
    dist.destroy_process_group()


def test_two_rank_reduction_and_independent_replicas():
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
    (_, max0, sum0, tok0), (_, max1, sum1, tok1) = res
    assert max0 == max1 == [11.0, 5.0, 1.0]
    assert sum0 == sum1 == [128.0, float(tok0 + tok1)]
    assert tok0 != tok1                      # different seeds: different trajectories per replica


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    m, s = bench.reduce_over_ranks(None, torch.device("cpu"), [3.0, 2.0], [7])
    assert m == [3.0, 2.0] and s == [7.0]
