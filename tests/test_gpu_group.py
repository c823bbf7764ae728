"""meteora_linear_forward_group on a B200: several MeteoRA linears that share x (q/k/v, gate/up of a decoder
block, each with its own gate and adapters, Sec. 3.2) against the CPU oracle, module by module."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import workloads
from .gpu_util import bf16_bound_ok, check_selection, clear_tokens, rel_l2, to_dev

pytestmark = pytest.mark.gpu


def make_group(T, d_in, d_outs, seed, dtype="bf16", N=28, k=2, b_std=0.3):
    """One workload per module; all take module 0's x."""
    ws = [workloads.make_workload(f"group/{m}", T=T, d_in=d_in, d_out=d, N=N, k=k, dtype=dtype, x_kind="rms",
                                  seed=seed + 31 * m, b_std=b_std) for m, d in enumerate(d_outs)]
    for w in ws[1:]:
        w.tensors["x"] = ws[0]["x"]
    return ws


def run_group(ws, workspace=None):
    x = to_dev(ws[0], "x")[0]
    W0s, As, Bs, Wgs = [], [], [], []
    for w in ws:
        W0, A, B, Wg = to_dev(w, "W0", "A", "B", "Wg")
        W0s.append(W0), As.append(A), Bs.append(B), Wgs.append(Wg)
    ys, routing = mb.meteora_linear_forward_group(x, W0s, As, Bs, Wgs, ws[0].k, ws[0].temperature,
                                                  workspace=workspace, return_routing=True)
    torch.cuda.synchronize()
    return ([y.float().cpu().numpy() for y in ys],
            [(i.cpu().numpy().copy(), w.cpu().numpy().copy()) for i, w in routing])


def check_group(ws, y_tol):
    ys, routing = run_group(ws)
    for w, y, (idx, wts) in zip(ws, ys, routing):
        o_idx, o_w, o_logits = oracle.gate_topk(w["x"], w["Wg"], w.k, w.temperature)
        clear = check_selection(idx, o_idx, o_logits, w.k)
        np.testing.assert_allclose(wts[clear], o_w[clear], rtol=1e-4, atol=1e-5)   # fp32 on shared bf16 inputs
        ref = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx, w.temperature)
        err = rel_l2(y, ref)
        assert err <= y_tol, (w.name, err)
        if w.dtype == "bf16":                                        # element by element: 5e-2 + one bf16 ulp of ref
            assert bf16_bound_ok(y, ref) <= 0.0, w.name
    return ys, routing


# q/k/v-like groups of a decode batch: one launch for the group.  Row-tile counts 5 + 2 + 3, a module that ends in
# the middle of a 128-row tile (1000 rows) followed by a small one, four modules, a contraction length that is
# no multiple of 64, and token counts from 1 to 256.
@pytest.mark.parametrize("d_in,d_outs,T", [
    (1024, (640, 256, 384), 1), (1024, (640, 256, 384), 37), (1024, (640, 256, 384), 128),
    (1536, (1000, 128), 200), (512, (256, 256, 128, 384), 16), (1096, (384, 640), 64), (1024, (2304, 768), 256),
])
def test_group_of_decode_modules_matches_oracle(d_in, d_outs, T):
    ws = make_group(T, d_in, d_outs, seed=6000 + T)
    assert mb.meteora_group_plan(T, d_in, list(d_outs), 28, 8, 2, torch.bfloat16) == 1
    ys1, r1 = check_group(ws, y_tol=1e-2)
    ys2, r2 = run_group(ws)
    for a, b in zip(ys1, ys2):
        np.testing.assert_array_equal(a, b)                          # counters re-armed, results reproducible


def test_group_agrees_with_separate_calls():
    ws = make_group(64, 1024, (640, 256, 384), seed=6100)
    ys, routing = run_group(ws)
    for w, y, (idx, _) in zip(ws, ys, routing):
        x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
        y1, i1, _ = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, return_routing=True)
        torch.cuda.synchronize()
        same = np.all(i1.cpu().numpy() == idx, axis=1)
        _, _, o_logits = oracle.gate_topk(w["x"], w["Wg"], w.k, w.temperature)
        assert np.all(same[clear_tokens(o_logits, w.k)])             # the two may differ only at near-ties
        assert same.mean() > 0.98
        assert rel_l2(y[same], y1.float().cpu().numpy()[same]) < 5e-3


def test_group_workspace_reused_across_calls():
    ws = make_group(8, 512, (256, 384), seed=6200)
    x = to_dev(ws[0], "x")[0]
    shape = mb.make_shape(8, 512, 256, 28, 8, 2, torch.bfloat16)
    import ctypes
    lib = mb.load_library()
    n = lib.meteora_group_workspace_bytes(ctypes.byref(shape), (ctypes.c_int * 2)(256, 384), 2)
    assert n > 0
    workspace = torch.zeros(n, dtype=torch.uint8, device="cuda")
    a, _ = run_group(ws, workspace)
    b, _ = run_group(ws, workspace)
    for u, v in zip(a, b):
        np.testing.assert_array_equal(u, v)
    assert mb.meteora_workspace_status(workspace) == 0


# What the one-launch kernel does not take runs module by module: a prefill batch, fp32 modules, and groups with
# so many row tiles that a CTA would finish more than two (gate/up of LLaMA3-8B: 224 tiles on 128 CTAs).
@pytest.mark.parametrize("T,dtype,d_outs,tol", [(300, "bf16", (128, 200), 1e-2), (20, "f32", (128, 200), 1e-4),
                                                (64, "bf16", (14336, 14336), 1e-2)])
def test_group_falls_back_module_by_module(T, dtype, d_outs, tol):
    N = 6 if dtype == "f32" else 28
    ws = make_group(T, 256, d_outs, seed=6300 + T, dtype=dtype, N=N)
    assert mb.meteora_group_plan(T, 256, list(d_outs), N, 8, 2, torch.float32 if dtype == "f32" else torch.bfloat16) == 0
    check_group(ws, y_tol=tol)


def test_group_argument_errors():
    ws = make_group(4, 256, (128, 128), seed=6400)
    x = to_dev(ws[0], "x")[0]
    W0, A, B, Wg = to_dev(ws[0], "W0", "A", "B", "Wg")
    with pytest.raises(mb.MeteoraError):
        mb.meteora_linear_forward_group(x, [W0] * 5, [A] * 5, [B] * 5, [Wg] * 5, 2)          # more than 4 modules
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(mb.MeteoraError):
        mb.meteora_linear_forward_group(x, [W0, W0], [A, A], [B, B], [Wg, Wg], 2, workspace=small)
