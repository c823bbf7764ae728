"""The N > 1 plumbing of bench.py on CPU: two `gloo` ranks.

The path shards by tokens / modules with replicated weights and no exchange step, so all a multi-rank run adds
is: seeds that differ per rank, a barrier, the maximum of the ranks' elapsed times, the whole-job token count,
and rank 0 alone printing.  None of that needs a GPU.
"""
import io
import os
import socket
import sys
from contextlib import redirect_stdout

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "WORLD_SIZE": str(world), "LOCAL_RANK": str(rank)})
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.rank_info() == (world, rank, rank)
        dist.barrier()
        slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")      # rank 1 is the slow shard
        seeds = [bench.module_seed(i, rank) for i in range(16)]
        gathered = [None] * world
        dist.all_gather_object(gathered, seeds)
        # the reference arm: only rank 0 works and prints
        buf = io.StringIO()
        printed = None
        if rank != 0:
            class A:                                                         # the fields run_reference reads
                tokens, steps, warmup, gpus = 1, 1, 1, world
            with redirect_stdout(buf):
                bench.run_reference(A)
            printed = buf.getvalue()
        out.put((rank, slowest, gathered, printed))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_take_the_slowest_time_and_disjoint_seeds():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=100) for _ in range(world))
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    for rank, slowest, gathered, printed in results:
        assert slowest == 15.0                                               # max over ranks, on every rank
        assert not (set(gathered[0]) & set(gathered[1]))                     # no module is timed twice
        if rank != 0:
            assert printed == ""                                             # only rank 0 prints


def test_whole_job_value_counts_every_rank():
    import bench

    one = bench.whole_job_value(16, 128, 1, 200, 400.0)
    assert one == pytest.approx(16 * 128 * 200 / 0.4)
    assert bench.whole_job_value(16, 128, 8, 200, 400.0) == pytest.approx(8 * one)
