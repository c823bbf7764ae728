"""meteora_pad_adapters: the rank of bf16 adapters zero-padded to a multiple of 8 once, instead of by every forward.

A rank-4 (or rank-12) bf16 layer runs on the tensor-core paths with A and B padded; the forward pads them into its
workspace on every call.  The adapters are fixed (Sec. 3.2), so a caller may pad them once and pass the padded
arrays with the padded rank.  The added rows of A and columns of B are zero, so the products do not change: the
output, the routing and the weights must be bit-identical to the forward that pads by itself, and both must match
the oracle on the ORIGINAL arrays."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import workloads

from .gpu_util import bf16_bound_ok, rel_l2, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", [
    dict(T=1, d_in=512, d_out=384, r=4),
    dict(T=30, d_in=512, d_out=384, r=4),
    dict(T=128, d_in=1024, d_out=640, r=4),
    dict(T=300, d_in=512, d_out=384, r=4),            # a prefill batch
    dict(T=40, d_in=256, d_out=256, r=12),            # padded to 16
])
def test_padding_once_gives_the_same_bits_as_padding_in_every_call(case):
    w = workloads.make_workload("pad", N=28, k=2, dtype="bf16", x_kind="normal", seed=4100 + case["T"], b_std=0.3,
                                **case)
    x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    y0, idx0, w0 = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, return_routing=True)
    y0, idx0, w0 = y0.clone(), idx0.clone(), w0.clone()
    A_pad, B_pad = mb.meteora_pad_adapters(A, B)
    r8 = (w.r + 7) // 8 * 8
    assert A_pad.shape == (w.N, r8, w.d_in) and B_pad.shape == (w.N, w.d_out, r8)
    assert torch.equal(A_pad[:, :w.r], A) and torch.equal(B_pad[:, :, :w.r], B)
    assert float(A_pad[:, w.r:].abs().max()) == 0.0 and float(B_pad[:, :, w.r:].abs().max()) == 0.0
    y1, idx1, w1 = mb.meteora_linear_forward(x, W0, A_pad, B_pad, Wg, w.k, return_routing=True)
    assert torch.equal(idx0, idx1) and torch.equal(w0, w1) and torch.equal(y0, y1)
    ref = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx1.cpu().numpy())
    y = y1.float().cpu().numpy()
    assert rel_l2(y, ref) <= 1e-2
    assert bf16_bound_ok(y, ref) <= 0.0


def test_padding_is_refused_where_the_library_does_not_pad():
    import ctypes
    lib = mb.load_library()
    A = torch.zeros(4, 8, 64, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(4, 32, 8, dtype=torch.bfloat16, device="cuda")
    assert mb.meteora_pad_adapters(A, B)[0] is A                       # rank 8: nothing to pad
    shape = mb.make_shape(0, 64, 32, 4, 8, 1, torch.bfloat16)
    assert lib.meteora_pad_adapters_bytes(ctypes.byref(shape), None, None) == 0
    assert lib.meteora_pad_adapters(A.data_ptr(), B.data_ptr(), ctypes.byref(shape), A.data_ptr(), B.data_ptr(),
                                    None) == -2                        # METEORA_ERR_UNSUPPORTED_SHAPE
    shape4 = mb.make_shape(0, 64, 32, 4, 4, 1, torch.bfloat16)
    assert lib.meteora_pad_adapters_bytes(ctypes.byref(shape4), None, None) == 8
    assert lib.meteora_pad_adapters(None, B.data_ptr(), ctypes.byref(shape4), A.data_ptr(), B.data_ptr(), None) == -1
