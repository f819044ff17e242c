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


def _handoff_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    H, D = 2, 8
    lens = np.array([5, 0, 17, 1], np.int32)
    if rank == 0:
        indptr = bench.handoff_plan(lens)
        # row r of trajectory t holds the value 1000 t + r in K and its negative in V
        k = torch.cat([1000.0 * t + torch.arange(int(n), dtype=torch.float32) for t, n in enumerate(lens)]).view(-1, 1, 1).expand(-1, H, D).contiguous()
        moved = bench.handoff_send(dist, 1, lens, k, -k)
        q.put((rank, int(moved), indptr.tolist()))
    else:
        got_lens, indptr, k, v = bench.handoff_recv(dist, 0, torch.device("cpu"), H, D, dtype=torch.float32)
        ok = list(got_lens) == list(lens) and tuple(k.shape) == (int(lens.sum()), H, D)
        for t in range(len(lens)):
            a, b = int(indptr[t]), int(indptr[t + 1])
            ok = ok and b - a == int(lens[t])
            ok = ok and bool(torch.equal(k[a:b, 0, 0], 1000.0 * t + torch.arange(b - a, dtype=torch.float32)))
            ok = ok and bool(torch.equal(v[a:b], -k[a:b]))
        q.put((rank, bool(ok), indptr.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_kv_handoff_exchange_between_two_ranks():
    """The wire part of the KV hand-off (Sec. 6.3) on CPU with gloo: lengths, then K and V rows, land in the receiver's
    own buffers with the indptr the receiver's append needs, and the byte count is the one the bench reports."""
    sys.path.insert(0, ROOT)
    import bench
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_handoff_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, moved, indptr0), (_, ok, indptr1) = res
    assert ok is True
    assert indptr0 == indptr1 == [0, 5, 5, 22, 23]
    assert moved == 2 * 23 * 2 * 8 * 4 == bench.handoff_bytes(23, 2, 8, elem_bytes=4)


def test_handoff_plan_refuses_more_rows_than_an_int32_holds():
    sys.path.insert(0, ROOT)
    import bench
    import pytest
    with pytest.raises(ValueError):
        bench.handoff_plan([2 ** 30, 2 ** 30])
    assert bench.handoff_plan([]).tolist() == [0]
