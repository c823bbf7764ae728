"""meteora_gate_backward on a B200 against the CPU oracle (Sec. 3.2 with Eq. 2, Eq. 3): the gradient of the gate
weights for the routing a forward produced."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import workloads
from .gpu_util import rel_l2, to_dev

pytestmark = pytest.mark.gpu

# fp32 accumulation of d_in- and d_out-long dot products on exactly shared inputs against fp64: 1e-3 leaves two
# orders of magnitude; the weights come from the GPU forward (fp32 softmax), the oracle recomputes its own.
TOL = {"bf16": 2e-3, "f32": 2e-4}


def dy_like(w, seed):
    rng = np.random.default_rng(seed)
    dy = rng.standard_normal((w.T, w.d_out)).astype(np.float32)
    return workloads.round_to_bf16(dy) if w.dtype == "bf16" else dy


@pytest.mark.parametrize("case", [
    dict(T=1, d_in=256, d_out=128, N=28, r=8, k=2, dtype="bf16"),
    dict(T=37, d_in=136, d_out=200, N=28, r=8, k=2, dtype="bf16"),               # ragged everything
    dict(T=300, d_in=512, d_out=384, N=28, r=8, k=2, dtype="bf16"),
    dict(T=64, d_in=256, d_out=256, N=12, r=16, k=4, dtype="bf16", temperature=3.0),
    dict(T=50, d_in=100, d_out=70, N=6, r=3, k=3, dtype="f32"),                  # nothing aligned, odd rank
    dict(T=40, d_in=128, d_out=96, N=64, r=8, k=8, dtype="f32"),                 # most adapters, most picks
    dict(T=20, d_in=64, d_out=64, N=5, r=8, k=1, dtype="bf16"),                  # top-1: zero gradient
    dict(T=1100, d_in=512, d_out=640, N=28, r=8, k=2, dtype="bf16"),             # dense shrinks on pairs of SMs
    dict(T=33, d_in=128, d_out=100, N=10, r=8, k=2, dtype="bf16"),               # d_out no multiple of 8: grouped shrink
    dict(T=130, d_in=1024, d_out=256, N=64, r=24, k=4, dtype="bf16"),            # 1536 stacked rows, rank 24
    dict(T=90, d_in=256, d_out=512, N=128, r=8, k=3, dtype="bf16"),              # 128 adapters
    dict(T=128, d_in=1024, d_out=640, N=28, r=8, k=2, dtype="bf16"),             # both shrinks in one launch, 16 / 10 k-steps
    dict(T=256, d_in=640, d_out=2048, N=28, r=8, k=2, dtype="bf16"),             # the same, the longer axis second
    dict(T=1024, d_in=512, d_out=512, N=28, r=8, k=2, dtype="bf16"),             # the most slots without buckets
    dict(T=1025, d_in=512, d_out=512, N=28, r=8, k=2, dtype="bf16"),             # the fewest with
    dict(T=16, d_in=4096, d_out=4096, N=28, r=8, k=2, dtype="bf16"),             # a decode batch at config 1's shape
])
def test_gate_backward_matches_oracle(case):
    kw = dict(case)
    w = workloads.make_workload("gate_bwd", x_kind="normal", seed=7700 + case["T"], b_std=0.3, **kw)
    x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    _, idx, wts = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, w.temperature, return_routing=True)
    idx, wts = idx.clone(), wts.clone()
    dy_np = dy_like(w, 5)
    dy = torch.from_numpy(dy_np).to("cuda").to(x.dtype)
    dWg, dlogit = mb.meteora_gate_backward(x, A, B, dy, idx, wts, w.temperature)
    dWg2, _ = mb.meteora_gate_backward(x, A, B, dy, idx, wts, w.temperature)
    # the adapters transposed beforehand (they are fixed while the gates train): the same numbers, bit for bit
    Bt = mb.meteora_transpose_adapters_b(B)
    assert torch.equal(Bt, B.transpose(1, 2).contiguous())
    dWg3, dlogit3 = mb.meteora_gate_backward(x, A, None, dy, idx, wts, w.temperature, Bt=Bt)
    torch.cuda.synchronize()
    assert torch.equal(dWg, dWg2)                                     # fixed summation order
    assert torch.equal(dWg, dWg3) and torch.equal(dlogit, dlogit3)
    o_dlogit, o_dWg = oracle.gate_backward(w["x"], w["A"], w["B"], w["Wg"], dy_np, idx.cpu().numpy(), w.temperature)
    if w.k == 1:
        assert float(dWg.abs().max()) == 0.0 and np.all(o_dWg == 0.0)
        return
    tol = TOL[w.dtype]
    assert rel_l2(dlogit.cpu().numpy(), o_dlogit) <= tol
    assert rel_l2(dWg.cpu().numpy(), o_dWg) <= tol
    untouched = np.setdiff1d(np.arange(w.N), np.unique(idx.cpu().numpy()))
    assert float(dWg[torch.from_numpy(untouched).long()].abs().max()) == 0.0 if untouched.size else True


def test_gate_backward_argument_errors():
    import ctypes
    lib = mb.load_library()
    shape = mb.make_shape(4, 64, 64, 8, 8, 2, torch.bfloat16)
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    p = buf.data_ptr()
    assert lib.meteora_gate_backward(p, p, p, p, p, p, ctypes.byref(shape), None, None, p, buf.numel(), None) == -1
    assert lib.meteora_gate_backward(p, p, p, p, p, p, ctypes.byref(shape), None, p, p, 64, None) == -4
    assert lib.meteora_gate_backward(p, p, None, p, p, p, ctypes.byref(shape), None, p, p, buf.numel(), None) == -1
    assert lib.meteora_gate_backward_bt(p, p, None, p, p, p, ctypes.byref(shape), None, p, p, buf.numel(), None) == -1
    assert lib.meteora_gate_backward_bt(p, p, p, p, p, p, ctypes.byref(shape), None, p, p, 64, None) == -4
    assert lib.meteora_transpose_adapters_b(None, ctypes.byref(shape), p, None) == -1
    assert lib.meteora_adapters_bt_bytes(ctypes.byref(shape)) == 8 * 64 * 8 * 2
