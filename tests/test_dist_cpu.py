"""The N>1 plumbing of the benchmark on CPU: two gloo ranks, no GPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1908_05460_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dist_util.env_rank() == (rank, world, rank)
        slow = dist_util.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
        b, e = dist_util.shard_batch(129, rank, world)
        counts = torch.tensor([e - b], dtype=torch.int64)
        dist.all_reduce(counts)
        out.put((rank, slow, (b, e), int(counts.item())))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_rank_and_cover_the_batch():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in results] == [15.0, 15.0]                   # both report the max
    assert results[0][2] == (0, 65) and results[1][2] == (65, 129)   # contiguous, disjoint, complete
    assert results[0][3] == 129


def test_single_process_fallbacks():
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.shard_batch(128, 0, 1) == (0, 128)
    assert [dist_util.shard_batch(10, r, 4) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]
    assert abs(dist_util.us_per_layer(1.9, 38, 1) - 50.0) < 1e-9
    assert abs(dist_util.us_per_layer(1.9, 38, 2) - 25.0) < 1e-9


def _dp_worker(rank, world, port, out):
    """Two ranks split a batch; each computes the filter gradient of its images (here with the CPU checker, standing
    in for a GPU rank's kernel output); one bucketed all-reduce must give the full-batch gradient for the exact and
    top-1 layers and leave the random-gradient layer alone."""
    import numpy as np
    from oracle import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(5)
        g = oracle.Shape(7, 3, 6, 6, 4, 3, 3, 1, 1, 1, 1)
        x = rng.standard_normal((g.n, g.c, g.h, g.w)); dy = rng.standard_normal((g.n, g.k, g.p, g.q))
        b, e = dist_util.shard_batch(g.n, rank, world)
        gs = oracle.Shape(e - b, g.c, g.h, g.w, g.k, g.r, g.s, 1, 1, 1, 1)
        mine_exact = torch.from_numpy(oracle.dw_exact(x[b:e], dy[b:e], gs)[0]).float()
        mine_top1 = torch.from_numpy(oracle.dw_top1(x[b:e], dy[b:e], gs)[0]).float()
        rand = torch.from_numpy(oracle.dw_random(g.k * g.c * g.r * g.s, 11, 1.0 / 128)).float()      # same on every rank
        dws = [mine_exact, rand.clone(), mine_top1]
        nbytes = dist_util.allreduce_dw_bucket(dws, [-1, 1, 2])
        full_exact = oracle.dw_exact(x, dy, g)[0]
        full_top1 = oracle.dw_top1(x, dy, g)[0]
        ok = (np.allclose(dws[0].numpy(), full_exact, atol=1e-4) and np.allclose(dws[2].numpy(), full_top1, atol=1e-4)
              and torch.equal(dws[1], rand) and nbytes == 2 * full_exact.size * 4)
        out.put((rank, bool(ok)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_data_parallel_dw_bucket_allreduce_gives_the_full_batch_gradient():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results == [(0, True), (1, True)]
    assert [dist_util.needs_allreduce(m) for m in (-1, 0, 1, 2, 3)] == [True, False, False, True, True]
