"""Column-parallel shards of one MeteoRA linear on a B200: the shards of 2 and 3 ranks, run one after the other on
the one GPU, give the rows of the whole layer's y and the same routing (the gate is replicated, Eq. 3)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import column_parallel as cp
from paper_2405_13053_b200 import workloads
from .gpu_util import rel_l2, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,world", [(8, 2), (64, 3), (600, 2)])
def test_shards_give_the_rows_of_the_whole_layer(T, world):
    w = workloads.make_workload("colpar", T=T, d_in=1024, d_out=1000, N=28, r=8, k=2, dtype="bf16", x_kind="rms",
                                seed=8800 + T, b_std=0.3)
    x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    y_full, idx_full, _ = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, w.temperature, return_routing=True)
    idx_full = idx_full.clone()
    parts = []
    for rank in range(world):
        W0s, Bs = cp.shard_module(W0, B, world, rank)
        o0, o1 = cp.shard_bounds(w.d_out, world, rank)
        assert W0s.shape[0] == o1 - o0 and Bs.shape[1] == o1 - o0
        y_local, idx, _ = mb.meteora_linear_forward(x, W0s, A, Bs, Wg, w.k, w.temperature, return_routing=True)
        assert torch.equal(idx, idx_full)                         # same gate, same stacked shrink: same picks
        parts.append(cp.column_parallel_forward(x, W0s, A, Bs, Wg, w.k, w.temperature))
        assert torch.equal(parts[-1], y_local)
    y = torch.cat(parts, dim=1)
    torch.cuda.synchronize()
    assert y.shape == y_full.shape
    ref = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx_full.cpu().numpy(), w.temperature)
    assert rel_l2(y.float().cpu().numpy(), ref) <= 1e-2
    # against the unsharded call: the split over CTAs differs, so sums may round differently by a bf16 ulp
    assert rel_l2(y.float().cpu().numpy(), y_full.float().cpu().numpy()) <= 4e-3
