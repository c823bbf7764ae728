"""The bounded device-side waits of the decode kernels, made to run out once, safely.

Every wait of the kernels (mbarrier phases, workspace counters) gives up after a limit, records it in the
workspace's status word, and the kernel drains and returns.  Here that limit is shortened to a few milliseconds
(knob wait_limit_us) and one counter of a workspace header is biased on the host so that it cannot reach its
target: the "all partials are in" wait of the CTAs that select then expires.  Nothing waits forever: every waiter in the
kernels is bounded by the same limit.  The call must return, meteora_workspace_status must report
METEORA_ERR_TIMEOUT, and after meteora_workspace_init the next call on that workspace must match the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import workloads

from .gpu_util import rel_l2, to_dev

pytestmark = pytest.mark.gpu

COUNTER_WORD = 16          # header word of the "stacked-shrink partials delivered" counter of all three decode kernels


@pytest.mark.parametrize("stream_kernel", [1, 0, "cluster"])
def test_an_expired_wait_is_reported_and_the_workspace_recovers(stream_kernel):
    w = workloads.make_workload("bounded", T=40, d_in=1024, d_out=640, dtype="bf16", x_kind="normal", seed=8800,
                                b_std=0.3)
    x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    ws = mb.alloc_workspace(shape)
    cluster = stream_kernel == "cluster"
    mb.meteora_set_tuning("stream", 1 if cluster else stream_kernel)
    mb.meteora_set_tuning("cluster_decode", 2 if cluster else 0)
    mb.meteora_set_tuning("wait_limit_us", 3000)
    try:
        assert ("cluster_decode" if cluster else "stream_decode" if stream_kernel else "fused_decode") in \
            mb.meteora_describe_plan(shape)
        ws[:4096].view(torch.int32)[COUNTER_WORD] = -1000000         # the counter can no longer reach its target
        torch.cuda.synchronize()
        mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, workspace=ws)
        torch.cuda.synchronize()                                     # the call returns: the wait gave up
        assert mb.meteora_workspace_status(ws) == -6                 # METEORA_ERR_TIMEOUT (and the header is cleared)
    finally:
        mb.meteora_set_tuning("wait_limit_us", 0)
    try:
        mb.meteora_workspace_init(ws)
        y, idx, _ = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, workspace=ws, return_routing=True)
        assert mb.meteora_workspace_status(ws) == 0
        ref = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx.cpu().numpy())
        assert rel_l2(y.float().cpu().numpy(), ref) <= 1e-2
        # and once more on the recovered workspace: the counters were left re-armed
        y2 = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, workspace=ws)
        assert mb.meteora_workspace_status(ws) == 0
        np.testing.assert_array_equal(y.float().cpu().numpy(), y2.float().cpu().numpy())
    finally:
        mb.meteora_set_tuning("stream", 1)
        mb.meteora_set_tuning("cluster_decode", 0)
