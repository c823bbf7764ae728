"""The entry point for callers that cannot allocate device memory (meteora_lora_delta_static).

Some users of this library call it from places where cudaMalloc is off limits (inside another framework's
allocator lock, in a serving loop with a frozen memory pool, from a binding that can only launch), so they
have no workspace to give to meteora_lora_delta.  The static variant keeps its scratch in a fixed array
inside the library instead.  This file checks, through the C ABI, that it returns what meteora_lora_delta
returns and what the CPU oracle computes for the same routing, on two calls in a row that share (and
overwrite) that array, and that it refuses problems larger than the array.  It is collected last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import workloads

pytestmark = pytest.mark.gpu


def _inputs(seed, T, d_in, d_out, dtype, N=28, r=8, k=2):
    w = workloads.make_workload("no_alloc", T=T, d_in=d_in, d_out=d_out, N=N, r=r, k=k, dtype=dtype, seed=seed,
                                b_std=0.3)
    dt = torch.float32 if dtype == "f32" else torch.bfloat16
    x, A, B, Wg = (torch.from_numpy(w[n]).cuda().to(dt) for n in ("x", "A", "B", "Wg"))
    idx, wts, _ = mb.meteora_gate_topk(x, Wg, k)
    _, offsets, perm = mb.meteora_route(idx, N)
    return (x, A, B, idx, wts, offsets, perm), w


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    first = _inputs(11, T=300, d_in=512, d_out=200, dtype="bf16")
    second = _inputs(12, T=77, d_in=136, d_out=328, dtype="f32", N=5, r=16, k=3)   # smaller: stale values stay behind
    for args, w in (first, second):
        expect = mb.meteora_lora_delta(*args)
        out = torch.full_like(expect, float("nan"))
        got = mb.meteora_lora_delta_static(*args, out=out)
        torch.cuda.synchronize()
        e, g = expect.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.linalg.norm(g - e) <= 1e-4 * np.linalg.norm(e)      # the tolerance of the LoRA-term parity tests
        assert np.linalg.norm(e) > 0
        # and against the oracle's LoRA term for the routing the GPU used (Eq. 2), same tolerance
        ref = oracle.lora_delta(w["x"], w["A"], w["B"], args[3].cpu().numpy(), args[4].cpu().numpy())
        assert np.linalg.norm(g - ref) <= 1e-4 * np.linalg.norm(ref)


def test_static_scratch_rejects_what_does_not_fit():
    T = mb.STATIC_SCRATCH_FLOATS // (2 * 8) + 1                      # one token too many for k=2, r=8
    too_big, _ = _inputs(13, T=T, d_in=64, d_out=32, dtype="bf16")
    with pytest.raises(mb.MeteoraError) as err:
        mb.meteora_lora_delta_static(*too_big)
    assert err.value.status == -2
    fits, _ = _inputs(14, T=T - 1, d_in=64, d_out=32, dtype="bf16")  # exactly at the limit still runs
    np.testing.assert_allclose(mb.meteora_lora_delta_static(*fits).cpu().numpy(),
                               mb.meteora_lora_delta(*fits).cpu().numpy(), rtol=1e-5, atol=1e-6)
