"""The multi-rank plan of bench.py on CPU ranks (gloo, world size 2): every rank builds the same
index recipe and draws its own query batch; the reported time is the maximum over ranks.  There is
no data-path collective to test: the search itself never leaves its GPU."""

import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        from ivfpq_inputs import generators as G
        cfg = bench.rank_config("c1", 64, rank).scaled(n=4000, ncomp=40, nlist=16, chunk=4000)
        spec = G.make_mixture(cfg, "cpu")
        q = G.queries(cfg, spec)
        means = spec.means.sum().reshape(1).double()
        qsum = q.sum().reshape(1).double()
        g_means = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        g_q = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(g_means, means)
        dist.all_gather(g_q, qsum)
        slow = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
        if rank == 0:
            out.put((float(g_means[0]), float(g_means[1]), float(g_q[0]), float(g_q[1]), slow))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_share_the_index_recipe_and_split_the_queries():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    m0, m1, q0, q1, slow = out.get()
    assert m0 == m1                      # same mixture (and so the same index) on both ranks
    assert q0 != q1                      # different query batches
    assert slow == 15.0                  # the job's time is the slowest rank's
