"""Column-parallel split of one MeteoRA linear (rows of W0 and of every B_i over the ranks; gate and shrink
replicated): the host logic on CPU.  Two `gloo` ranks each run the oracle on their shard as the single-rank
forward; the gathered result must equal the oracle on the whole layer exactly, because Eq. 2 is row-wise in W0
and B_i and the routing (Eq. 3) does not depend on the shard."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_13053_b200 import column_parallel as cp  # noqa: E402


@pytest.mark.parametrize("d_out", [1, 127, 128, 129, 1000, 4096, 14336])
@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_shard_bounds_cover_the_rows_once_in_whole_tiles(d_out, world):
    bounds = [cp.shard_bounds(d_out, world, r) for r in range(world)]
    assert bounds[0][0] == 0 and bounds[-1][1] == d_out
    for (a0, a1), (b0, b1) in zip(bounds, bounds[1:]):
        assert a1 == b0 and a0 <= a1
    for o0, o1 in bounds:
        assert o0 % cp.ROW_TILE == 0 and (o1 % cp.ROW_TILE == 0 or o1 == d_out)
    widths = [b - a for a, b in bounds]
    assert max(widths) - min(widths) <= cp.ROW_TILE                     # tiles dealt evenly


def test_shard_bounds_rejects_bad_requests():
    with pytest.raises(ValueError):
        cp.shard_bounds(128, 2, 2)
    with pytest.raises(ValueError):
        cp.shard_bounds(128, 0, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle_forward(x, W0, A, B, Wg, k, temperature=1.0):
    import oracle
    y, _, _ = oracle.linear_forward(x.numpy(), W0.numpy(), A.numpy(), B.numpy(), Wg.numpy(), k, temperature)
    return torch.from_numpy(y.astype(np.float32))


def _worker(rank, world, port, d_out, out):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "WORLD_SIZE": str(world)})
    from paper_2405_13053_b200 import workloads
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = workloads.make_workload("colpar", T=9, d_in=64, d_out=d_out, N=6, r=4, k=2, dtype="f32", seed=77)
        x, W0, A, B, Wg = (torch.from_numpy(w[n]) for n in ("x", "W0", "A", "B", "Wg"))
        W0s, Bs = cp.shard_module(W0, B, world, rank)
        y_local = cp.column_parallel_forward(x, W0s, A, Bs, Wg, w.k, w.temperature, forward=_oracle_forward)
        y = cp.column_parallel_forward(x, W0s, A, Bs, Wg, w.k, w.temperature, d_out=d_out, gather=True,
                                       forward=_oracle_forward)
        out.put((rank, tuple(y_local.shape), y.numpy()))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(180)
@pytest.mark.parametrize("d_out", [300, 100])     # 3 row tiles over 2 ranks (uneven widths); 1 tile: rank 0 owns nothing
def test_two_ranks_gather_the_oracle_result_of_the_whole_layer(d_out):
    import oracle
    from paper_2405_13053_b200 import workloads
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, d_out, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=150) for _ in range(world))
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    w = workloads.make_workload("colpar", T=9, d_in=64, d_out=d_out, N=6, r=4, k=2, dtype="f32", seed=77)
    y_full, _, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], w.k, w.temperature)
    widths = [b - a for a, b in (cp.shard_bounds(d_out, world, r) for r in range(world))]
    for rank, local_shape, y in results:
        assert local_shape == (9, widths[rank])
        np.testing.assert_array_equal(y, y_full.astype(np.float32))
