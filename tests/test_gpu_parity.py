"""GPU parity: every entry point of the C ABI against the CPU oracle, element by element, on the same
seeded inputs.  Tolerances (stated where used):
  - indices, counts, offsets, perm: bit-exact (selections only where the logit gap exceeds 1e-3);
  - fp32 layers: relative L2 <= 1e-4 (measured ~1e-6);
  - bf16 layers: y relative L2 <= 1e-2 and, element by element, |y - ref| <= 5e-2 + 2^-8 |ref| (the absolute
    bound plus one bf16 ulp of the reference, so that large outputs are not excused wholesale: a wrong row
    tile, a dropped pick or a stale partial tile breaks it); fp32 intermediates (routing weights, delta)
    <= 1e-4, since both sides read the same bf16 values and the GPU accumulates in fp32.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_13053_b200 import binding as mb
from paper_2405_13053_b200 import workloads

from .gpu_util import bf16_bound_ok, check_selection, clear_tokens, max_abs, rel_l2, to_dev

pytestmark = pytest.mark.gpu


def wl(T, d_in, d_out, N=5, r=8, k=2, dtype="bf16", seed=1, b_std=0.3, x_kind="normal", temperature=1.0):
    return workloads.make_workload("t", T=T, d_in=d_in, d_out=d_out, N=N, r=r, k=k, dtype=dtype, x_kind=x_kind,
                                   seed=seed, b_std=b_std, temperature=temperature)


# ----------------------------------------------------------------------------------------- gate + top-k
GATE_CASES = [
    dict(T=64, d_in=256, d_out=8, N=4, k=2, dtype="f32"),
    dict(T=37, d_in=136, d_out=8, N=28, k=2, dtype="bf16"),
    dict(T=5, d_in=23, d_out=8, N=7, k=3, dtype="f32"),          # d_in not a multiple of 8: scalar loads
    dict(T=19, d_in=72, d_out=8, N=40, k=8, dtype="bf16"),       # more than 32 adapters, k = 8
    dict(T=9, d_in=64, d_out=8, N=64, k=1, dtype="f32"),         # top-1
    dict(T=11, d_in=48, d_out=8, N=6, k=6, dtype="bf16"),        # k = N
    dict(T=21, d_in=128, d_out=8, N=128, k=8, dtype="f32"),      # the most adapters: four logits per lane
    dict(T=17, d_in=256, d_out=8, N=100, k=4, dtype="bf16"),     # the last lanes' fourth logit is out of range
    dict(T=1, d_in=4096, d_out=8, N=28, k=2, dtype="bf16"),
    dict(T=300, d_in=512, d_out=8, N=28, k=2, dtype="bf16", temperature=15.0),
    dict(T=128, d_in=4096, d_out=8, N=28, k=2, dtype="bf16"),     # long rows: 8 warps share a token's contraction axis
    dict(T=1101, d_in=1024, d_out=8, N=28, k=2, dtype="bf16"),    # ... and from 1024 tokens up 4 tokens per block, ragged
    dict(T=70, d_in=1536, d_out=8, N=128, k=8, dtype="f32"),      # ... fp32, the most adapters
]


@pytest.mark.parametrize("case", GATE_CASES, ids=lambda c: f"T{c['T']}d{c['d_in']}N{c['N']}k{c['k']}{c['dtype']}")
def test_gate_topk_matches_oracle(case):
    w = wl(**case)
    x, Wg = to_dev(w, "x", "Wg")
    idx, wts, logits = mb.meteora_gate_topk(x, Wg, w.k, w.temperature, want_logits=True)
    torch.cuda.synchronize()
    o_idx, o_w, o_logits = oracle.gate_topk(w["x"], w["Wg"], w.k, w.temperature)
    np.testing.assert_allclose(logits.cpu().numpy(), o_logits, rtol=1e-4, atol=1e-5)
    clear = check_selection(idx.cpu().numpy(), o_idx, o_logits, w.k)
    assert clear.mean() > 0.9
    g_w = wts.cpu().numpy()
    np.testing.assert_allclose(g_w[clear], o_w[clear], rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(g_w.sum(axis=1), 1.0, atol=1e-6)      # Eq. 3: weights sum to one
    if w.k == 1:
        assert np.all(g_w == 1.0)


def test_gate_ties_resolve_to_lower_index():
    w = wl(T=33, d_in=64, d_out=8, N=40, k=3, dtype="f32")
    Wg = np.zeros_like(w["Wg"])
    Wg[[3, 17, 35, 38], 0] = 7.0                                     # four exactly equal logits
    x = w["x"].copy()
    x[:, 0] = 1.0
    idx, wts, _ = mb.meteora_gate_topk(torch.from_numpy(x).cuda(), torch.from_numpy(Wg).cuda(), 3)
    o_idx, o_w, _ = oracle.gate_topk(x, Wg, 3)
    np.testing.assert_array_equal(idx.cpu().numpy(), o_idx)
    np.testing.assert_array_equal(o_idx[0], [3, 17, 35])
    np.testing.assert_allclose(wts.cpu().numpy(), o_w, rtol=1e-6)


# ----------------------------------------------------------------------------------------- routing
def random_idx(T, k, N, seed, skew=False):
    rng = np.random.default_rng(seed)
    idx = np.stack([rng.permutation(N)[:k] for _ in range(T)]).astype(np.int32) if T else np.zeros((0, k), np.int32)
    if skew and T > 4:
        hot = rng.permutation(N)[:max(k, 3)]
        idx[: 3 * T // 4] = np.stack([rng.permutation(hot)[:k] for _ in range(3 * T // 4)])
    return idx


@pytest.mark.parametrize("T,k,N,skew", [(0, 2, 4, False), (1, 1, 1, False), (1, 2, 28, False), (64, 2, 4, False),
                                         (511, 2, 28, True), (512, 2, 28, True), (513, 2, 28, False),
                                         (1500, 3, 64, True), (8192, 2, 28, True), (100, 8, 8, False)])
def test_route_is_bit_exact(T, k, N, skew):
    idx = random_idx(T, k, N, seed=T + k + N, skew=skew)
    counts, offsets, perm = mb.meteora_route(torch.from_numpy(idx).cuda(), N)
    torch.cuda.synchronize()
    o_counts, o_offsets, o_perm = oracle.route(idx, N)
    np.testing.assert_array_equal(counts.cpu().numpy(), o_counts)
    np.testing.assert_array_equal(offsets.cpu().numpy(), o_offsets)
    np.testing.assert_array_equal(perm.cpu().numpy(), o_perm)


def test_route_all_tokens_to_one_adapter():
    idx = np.tile(np.array([[5, 2]], np.int32), (2000, 1))
    counts, offsets, perm = mb.meteora_route(torch.from_numpy(idx).cuda(), 28)
    o = oracle.route(idx, 28)
    for g, e in zip((counts, offsets, perm), o):
        np.testing.assert_array_equal(g.cpu().numpy(), e)


# ----------------------------------------------------------------------------------------- LoRA term
DELTA_CASES = [
    dict(T=64, d_in=256, d_out=256, N=4, r=8, k=2, dtype="f32"),
    dict(T=77, d_in=136, d_out=200, N=28, r=8, k=2, dtype="bf16"),
    dict(T=13, d_in=23, d_out=19, N=5, r=3, k=2, dtype="f32"),       # nothing aligned: scalar paths
    dict(T=40, d_in=4096, d_out=320, N=28, r=16, k=2, dtype="bf16"),  # rank 16, several shared-memory chunks
    dict(T=9, d_in=2304, d_out=64, N=6, r=12, k=3, dtype="f32"),      # rank not a multiple of 8
    dict(T=300, d_in=512, d_out=96, N=28, r=8, k=1, dtype="bf16", x_kind="clusters"),
]


@pytest.mark.parametrize("case", DELTA_CASES, ids=lambda c: f"T{c['T']}d{c['d_in']}o{c['d_out']}r{c['r']}{c['dtype']}")
def test_lora_delta_matches_oracle(case):
    w = wl(**case)
    o_idx, o_w, _ = oracle.gate_topk(w["x"], w["Wg"], w.k)
    w32 = o_w.astype(np.float32)
    x, A, B = to_dev(w, "x", "A", "B")
    idx = torch.from_numpy(o_idx).cuda()
    wts = torch.from_numpy(w32).cuda()
    _, offsets, perm = mb.meteora_route(idx, w.N)
    delta = mb.meteora_lora_delta(x, A, B, idx, wts, offsets, perm)
    torch.cuda.synchronize()
    ref = oracle.lora_delta(w["x"], w["A"], w["B"], o_idx, w32)
    assert rel_l2(delta.cpu().numpy(), ref) <= 1e-4                  # fp32 accumulate on identical inputs
    assert np.linalg.norm(ref) > 0


def test_lora_delta_with_empty_adapters_and_single_hot_adapter():
    w = wl(T=50, d_in=128, d_out=72, N=28, r=8, k=2, dtype="bf16")
    o_idx = np.tile(np.array([[9, 27]], np.int32), (50, 1))          # 26 adapters receive no token
    w32 = np.tile(np.array([[0.75, 0.25]], np.float32), (50, 1))
    x, A, B = to_dev(w, "x", "A", "B")
    idx = torch.from_numpy(o_idx).cuda()
    _, offsets, perm = mb.meteora_route(idx, w.N)
    delta = mb.meteora_lora_delta(x, A, B, idx, torch.from_numpy(w32).cuda(), offsets, perm)
    ref = oracle.lora_delta(w["x"], w["A"], w["B"], o_idx, w32)
    assert rel_l2(delta.cpu().numpy(), ref) <= 1e-4


@pytest.fixture
def cooperative_decode_kernel():
    """The earlier one-launch decode kernel (cooperative launch, one CTA per SM) instead of the streamed one."""
    mb.meteora_set_tuning("stream", 0)
    yield
    mb.meteora_set_tuning("stream", 1)


# ----------------------------------------------------------------------------------------- whole layer
# Routing weights of the fused paths against the oracle: fp32 logits from the stacked tensor-core product (bf16
# inputs, fp32 accumulation, slices of the contraction axis added in fp32) differ from the fp64 logits by a few
# 1e-6, and a softmax weight moves by at most a quarter of the logit error.
W_RTOL, W_ATOL = 1e-4, 1e-5


def run_forward(w, **kw):
    x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, x.dtype, w.temperature)
    ws = mb.alloc_workspace(shape)
    y, idx, wts = mb.meteora_linear_forward(x, W0, A, B, Wg, w.k, w.temperature, workspace=ws, return_routing=True)
    assert mb.meteora_workspace_status(ws) == 0
    return y.float().cpu().numpy(), idx.cpu().numpy().copy(), wts.cpu().numpy().copy()


def check_forward(w, y_tol, abs_tol=None, tokens=None):
    """Compare the fused forward with the oracle; `tokens` restricts the y comparison to sampled rows.
    The routing (selection and weights) is always checked on every token."""
    y, idx, wts = run_forward(w)
    o_idx, o_w, o_logits = oracle.gate_topk(w["x"], w["Wg"], w.k, w.temperature)
    clear = check_selection(idx, o_idx, o_logits, w.k)
    np.testing.assert_allclose(wts[clear], o_w[clear], rtol=W_RTOL, atol=W_ATOL)
    np.testing.assert_allclose(wts.sum(axis=1), 1.0, atol=1e-6)
    sel = np.arange(w.T) if tokens is None else np.asarray(tokens)
    ref = oracle.linear_forward_routed(w["x"][sel], w["W0"], w["A"], w["B"], w["Wg"], idx[sel], w.temperature)
    err = rel_l2(y[sel], ref)
    assert err <= y_tol, err
    if w.dtype == "bf16":
        excess = bf16_bound_ok(y[sel], ref)
        assert excess <= 0.0, excess
    if abs_tol is not None:
        assert max_abs(y[sel], ref) <= abs_tol
    return y, idx, err


def assert_same_outside_the_band(w, i0, i1):
    """Two paths may pick differently only where the oracle's logits are within GAP of a tie."""
    _, _, o_logits = oracle.gate_topk(w["x"], w["Wg"], w.k, w.temperature)
    clear = clear_tokens(o_logits, w.k)
    same = np.all(i0 == i1, axis=1)
    assert np.all(same[clear]), np.nonzero(clear & ~same)[0]
    return same


def test_config0_fp32():
    w = workloads.config0()
    _, _, err = check_forward(w, y_tol=1e-4)
    assert err < 1e-5


FORWARD_CASES = [
    dict(T=13, d_in=24, d_out=20, N=5, r=3, k=2, dtype="f32"),                    # plain path, nothing aligned
    dict(T=70, d_in=100, d_out=130, N=28, r=8, k=2, dtype="f32"),
    dict(T=33, d_in=60, d_out=50, N=6, r=4, k=2, dtype="bf16"),                   # bf16 on the plain path (r % 8 != 0)
    dict(T=37, d_in=136, d_out=200, N=28, r=8, k=2, dtype="bf16"),                # tensor-core path, ragged everywhere
    dict(T=1, d_in=512, d_out=384, N=28, r=8, k=2, dtype="bf16"),
    dict(T=129, d_in=1024, d_out=256, N=28, r=8, k=2, dtype="bf16"),
    dict(T=300, d_in=2048, d_out=640, N=28, r=8, k=2, dtype="bf16"),              # two token tiles, ragged tail
    dict(T=50, d_in=512, d_out=128, N=40, r=16, k=3, dtype="bf16"),               # 40 adapters, rank 16, top-3
    dict(T=20, d_in=256, d_out=128, N=8, r=8, k=1, dtype="bf16"),                 # top-1
    dict(T=40, d_in=512, d_out=256, N=28, r=32, k=4, dtype="bf16"),               # rank 32, top-4, decode batch
    dict(T=30, d_in=512, d_out=384, N=28, r=4, k=2, dtype="bf16"),                # rank 4: adapters zero-padded to 8
    dict(T=300, d_in=1024, d_out=256, N=28, r=8, k=2, dtype="bf16"),              # short prefill grid: two CTAs per 128-token tile
    dict(T=700, d_in=8192, d_out=512, N=28, r=8, k=2, dtype="bf16"),              # long axis: two CTAs per 256-token tile
    dict(T=300, d_in=256, d_out=256, N=12, r=12, k=3, dtype="bf16"),              # rank 12 -> 16, prefill batch
    dict(T=600, d_in=512, d_out=200, N=28, r=64, k=2, dtype="bf16"),              # rank 64 prefill, d_out % 8 == 0 only
    dict(T=24, d_in=256, d_out=136, N=4, r=8, k=4, dtype="bf16", temperature=20.0),  # k = N with temperature
    dict(T=26, d_in=96, d_out=72, N=128, r=4, k=8, dtype="f32"),                  # 128 adapters on the plain path
    dict(T=300, d_in=512, d_out=256, N=128, r=8, k=2, dtype="bf16"),              # 128 adapters: 1024 stacked rows + a gate tile
]


@pytest.mark.parametrize("case", FORWARD_CASES,
                         ids=lambda c: f"T{c['T']}d{c['d_in']}o{c['d_out']}N{c['N']}r{c['r']}k{c['k']}{c['dtype']}")
def test_forward_small_shapes(case):
    w = wl(**case)                                                   # B ~ N(0, 0.3): the LoRA term is as large as the base
    if w.dtype == "f32":
        check_forward(w, y_tol=1e-4)
    else:
        check_forward(w, y_tol=1e-2)


@pytest.mark.parametrize("T", workloads.CONFIG1_T)
def test_config1_decode_shapes(T):
    w = workloads.config1(T)
    y, idx, err = check_forward(w, y_tol=1e-2, abs_tol=5e-2)                # at |y| ~ 1.3 the plain bound holds too
    assert err < 5e-3                                                # one bf16 rounding of y: ~2^-9 per element


def test_zero_B_is_exactly_the_base_product_and_delta_is_visible():
    w = wl(T=96, d_in=1024, d_out=384, N=28, r=8, k=2, dtype="bf16", b_std=0.3)
    y, idx, _ = run_forward(w)
    w0 = wl(T=96, d_in=1024, d_out=384, N=28, r=8, k=2, dtype="bf16", b_std=0.3)
    w0.tensors["B"] = np.zeros_like(w["B"])
    y0, _, _ = run_forward(w0)
    base = w["x"].astype(np.float64) @ w["W0"].astype(np.float64).T
    assert rel_l2(y0, base) < 5e-3                                   # Eq. 2 with B = 0
    o_idx, o_w, _ = oracle.gate_topk(w["x"], w["Wg"], w.k)
    ref_delta = oracle.lora_delta(w["x"], w["A"], w["B"], idx, o_w.astype(np.float32))
    assert np.linalg.norm(ref_delta) > 0.3 * np.linalg.norm(base)    # the LoRA term is not hidden under the base
    assert rel_l2(y - y0, ref_delta) <= 1e-2


def test_forward_is_deterministic():
    w = workloads.config1(32)
    y1, i1, w1 = run_forward(w)
    y2, i2, w2 = run_forward(w)
    np.testing.assert_array_equal(y1, y2)
    np.testing.assert_array_equal(i1, i2)
    np.testing.assert_array_equal(w1, w2)


def test_tensor_core_and_plain_paths_agree():
    w = wl(T=45, d_in=512, d_out=264, N=28, r=8, k=2, dtype="bf16")
    y_tc, i_tc, _ = run_forward(w)
    mb.meteora_set_tuning("force_simt", 1)
    try:
        y_simt, i_simt, _ = run_forward(w)
    finally:
        mb.meteora_set_tuning("force_simt", 0)
    same = assert_same_outside_the_band(w, i_tc, i_simt)
    assert same.mean() > 0.95
    assert rel_l2(y_tc[same], y_simt[same]) < 5e-3


@pytest.mark.parametrize("splits,stages", [(1, 2), (2, 3), (3, 4), (8, 2)])
def test_split_k_cluster_sizes_agree_with_oracle(splits, stages):
    w = wl(T=40, d_in=1536, d_out=200, N=28, r=8, k=2, dtype="bf16")
    mb.meteora_set_tuning("splits", splits)
    mb.meteora_set_tuning("stages", stages)
    try:
        check_forward(w, y_tol=1e-2)
    finally:
        mb.meteora_set_tuning("splits", 0)
        mb.meteora_set_tuning("stages", 0)


# (d_in, d_out) chosen so that the unit ranges of the main CTAs fall every way they can: many CTAs per row tile
# (640), a ragged last tile (1000), a contraction length that is no multiple of 64 (1096: plain 2-D tensor
# maps, one k-step per stage), ranges that straddle two tiles (4224 = 33 tiles over 128 CTAs), more tiles than
# half the CTAs (9000 = 71 tiles), with the "splits" knob capping the CTAs per tile, one CTA per tile, and layers
# with several row tiles per CTA (40000 and 60000 rows: 313 and 469 tiles on 128 CTAs).
@pytest.mark.parametrize("d_in,d_out,T,per_tile", [
    (1024, 640, 1, 0), (1024, 640, 8, 0), (1024, 640, 100, 0), (1024, 640, 256, 0),
    (1536, 1000, 37, 0), (1096, 768, 16, 0), (2048, 4224, 5, 0), (2048, 4224, 128, 0),
    (512, 9000, 24, 0), (1024, 1280, 64, 1), (1024, 1280, 200, 3),
    (128, 40000, 4, 0), (128, 60000, 70, 0),     # more row tiles than CTAs: unit ranges over three and four tiles
])
def test_single_launch_decode_kernel_matches_oracle(d_in, d_out, T, per_tile, cooperative_decode_kernel):
    # one kernel per call: base product + stacked shrink + selection + LoRA expand
    w = workloads.make_workload("fused", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="rms",
                                seed=50 + T + d_out, b_std=0.3)
    mb.meteora_set_tuning("splits", per_tile)
    mb.meteora_set_tuning("fused", 2)                                # 2: also where the three launches are the default
    try:
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        assert "fused_decode" in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
        y1, i1, _ = run_forward(w)
        y2, i2, _ = run_forward(w)
        np.testing.assert_array_equal(y1, y2)                        # counters re-armed, result reproducible
        np.testing.assert_array_equal(i1, i2)
    finally:
        mb.meteora_set_tuning("splits", 0)
        mb.meteora_set_tuning("fused", 1)


# Adapter counts that change the layout of the stacked shrink: Wg behind A's only tile (N = 4), Wg in a tile of
# its own (N = 16: A fills its tile), three A tiles with Wg behind 8 rows (N = 33, logits beyond one warp).
# ... and ranks above 8 (16-byte words per B row: 2, 3, 4), which also change the number of stacked-shrink tiles.
@pytest.mark.parametrize("N,k,T,r", [(4, 2, 9, 8), (16, 4, 40, 8), (33, 3, 130, 8), (2, 1, 3, 8),
                                     (28, 2, 20, 16), (28, 2, 128, 32), (10, 3, 64, 24),
                                     (128, 2, 64, 8), (100, 8, 7, 8), (72, 4, 128, 16)])   # more than 64 adapters
def test_single_launch_decode_kernel_adapter_counts(N, k, T, r, cooperative_decode_kernel):
    w = workloads.make_workload("fused_n", T=T, d_in=768, d_out=896, N=N, k=k, r=r, dtype="bf16", x_kind="normal",
                                seed=900 + N + r, b_std=0.3)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    assert "fused_decode" in mb.meteora_describe_plan(shape)
    check_forward(w, y_tol=1e-2)


# Planner choices of the decode kernel forced the other way: the aux CTAs' head start (none, the counter wait,
# a long timed one), how the units are dealt (even ranges over all free SMs: 5 row tiles on 128 CTAs share tiles
# unevenly; whole tiles per CTA group), and fewer or more aux CTAs (slices of the stacked shrink).  The result
# must not depend on any of them beyond the rounding order of the fp32 sums.
@pytest.mark.parametrize("knob,value", [("no_hold", 1), ("no_hold", 64), ("no_hold", 5000), ("unit_split", 1),
                                        ("unit_split", 2), ("aux_ctas", 4), ("aux_ctas", 40), ("kc", 1), ("stages", 2),
                                        ("hold_after", 1), ("hold_after", 3), ("narrow_select", -1),
                                        ("narrow_select", 1)])
def test_decode_kernel_planner_choices_do_not_change_the_result(knob, value, cooperative_decode_kernel):
    w = workloads.make_workload("fused_knobs", T=70, d_in=1024, d_out=640, dtype="bf16", x_kind="normal", seed=1234,
                                b_std=0.3)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    y0, i0, _ = run_forward(w)
    mb.meteora_set_tuning(knob, value)
    try:
        assert "fused_decode" in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
        y1, i1, _ = run_forward(w)
    finally:
        mb.meteora_set_tuning(knob, 0)
    same = assert_same_outside_the_band(w, i0, i1)   # another slicing of the shrink may flip a near-tie of two logits
    assert same.mean() > 0.97
    assert rel_l2(y1[same], y0[same]) < 4e-3


# The decode kernel's selection has two forms (the whole stacked row of a token in one round trip, or the logits
# first and then only the picks' shrink values); both add the partial copies in slice order, so routing, weights and
# y must agree bit for bit, for one pick and several, rank 8 and above, few and many adapters.
@pytest.mark.parametrize("T,N,r,k", [(70, 28, 8, 2), (9, 28, 8, 1), (40, 40, 16, 3), (33, 128, 8, 4), (20, 28, 32, 8)])
def test_both_forms_of_the_selection_agree_bit_for_bit(T, N, r, k, cooperative_decode_kernel):
    w = workloads.make_workload("select_forms", T=T, d_in=1024, d_out=384, N=N, r=r, k=k, dtype="bf16",
                                x_kind="normal", seed=5200 + T, b_std=0.3)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    out = {}
    try:
        for form in (-1, 1):
            mb.meteora_set_tuning("narrow_select", form)
            assert "fused_decode" in mb.meteora_describe_plan(shape)
            out[form] = run_forward(w)
    finally:
        mb.meteora_set_tuning("narrow_select", 0)
    for a, b in zip(out[-1], out[1]):
        np.testing.assert_array_equal(a, b)
    check_forward(w, y_tol=1e-2)


# Back-to-back decode calls in which every call reads what the call before it wrote (y of layer i is x of layer
# i + 1, as in a decoder stack), launched without any synchronisation in between.  The decode kernel is launched
# with programmatic stream serialization (its CTAs may move onto an SM as soon as the previous kernel's CTA has
# left it): it must not touch the previous result before that kernel has completed.  The chain with the
# attribute and without it (knob pdl_decode) must agree bit for bit, and so must a repeat.
@pytest.mark.parametrize("stream_kernel", [1, 0])
@pytest.mark.parametrize("T,d", [(40, 512), (130, 1024), (128, 2048)])
def test_dependent_decode_calls_back_to_back(T, d, stream_kernel):
    layers = [workloads.make_workload(f"stack{i}", T=T, d_in=d, d_out=d, dtype="bf16", x_kind="normal",
                                      seed=4100 + 7 * i, b_std=0.3) for i in range(4)]
    dev = [to_dev(w, "W0", "A", "B", "Wg") for w in layers]
    x0 = to_dev(layers[0], "x")[0]
    shape = mb.make_shape(T, d, d, layers[0].N, layers[0].r, layers[0].k, torch.bfloat16)
    mb.meteora_set_tuning("stream", stream_kernel)
    try:
        plan = mb.meteora_describe_plan(shape)
    finally:
        mb.meteora_set_tuning("stream", 1)
    # the streamed kernel takes up to 128 tokens: its CTAs are resident, and load weights, while the call ahead runs
    assert ("stream_decode" if stream_kernel and T <= 128 else "fused_decode") in plan
    wss = [mb.alloc_workspace(shape) for _ in layers]

    def run_stack():
        h = x0
        for (W0, A, B, Wg), ws in zip(dev, wss):
            h = mb.meteora_linear_forward(h, W0, A, B, Wg, layers[0].k, workspace=ws)
        torch.cuda.synchronize()
        for ws in wss:
            assert mb.meteora_workspace_status(ws) == 0
        return h.float().cpu().numpy()

    results = {}
    try:
        mb.meteora_set_tuning("stream", stream_kernel)
        for pdl in (1, 0, 1):
            mb.meteora_set_tuning("pdl_decode", pdl)
            results.setdefault(pdl, []).append(run_stack())
    finally:
        mb.meteora_set_tuning("pdl_decode", 1)
        mb.meteora_set_tuning("stream", 1)
    assert np.all(np.isfinite(results[1][0]))
    np.testing.assert_array_equal(results[1][0], results[0][0])
    np.testing.assert_array_equal(results[1][0], results[1][1])
    # and layer 0 alone against the oracle, as everywhere else
    y0 = mb.meteora_linear_forward(x0, *dev[0], layers[0].k, workspace=wss[0], return_routing=True)
    ref = oracle.linear_forward_routed(layers[0]["x"], layers[0]["W0"], layers[0]["A"], layers[0]["B"], layers[0]["Wg"],
                                       y0[1].cpu().numpy())
    assert rel_l2(y0[0].float().cpu().numpy(), ref) <= 1e-2


# ----------------------------------------------------------------------------------------- streamed decode kernel
# The decode kernel whose CTAs share an SM two at a time (up to 128 tokens).  Shapes chosen for every way its work
# splits: one CTA per row tile (1280 rows with splits = 1; 9000 rows = 71 tiles), several CTAs per tile with even
# row slices (2, 4, 8) and uneven ones (3, 5, 6, 7: slices of 10 / 11 groups of 4 rows), a ragged last tile (1000
# rows, 1001 rows: scalar stores), k-steps that do not divide by the CTAs per tile (1088 = 17 k-steps), one token,
# a token count that is no multiple of 16, and the full 128.
@pytest.mark.parametrize("d_in,d_out,T,per_tile", [
    (1024, 640, 1, 0), (1024, 640, 8, 0), (1024, 640, 100, 0), (1024, 640, 128, 0),
    (1536, 1000, 37, 0), (1088, 768, 16, 0), (2048, 4224, 5, 0), (2048, 4224, 128, 0),
    (512, 9000, 24, 0), (1024, 1280, 64, 1), (1024, 1280, 128, 2), (1024, 1280, 77, 3), (1024, 1001, 50, 5),
    (1024, 384, 128, 6), (1024, 384, 19, 7), (4096, 1024, 128, 0),
])
def test_streamed_decode_kernel_matches_oracle(d_in, d_out, T, per_tile):
    w = workloads.make_workload("stream", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="rms",
                                seed=150 + T + d_out, b_std=0.3)
    mb.meteora_set_tuning("splits", per_tile)
    try:
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        plan = mb.meteora_describe_plan(shape)
        assert "stream_decode" in plan
        if per_tile:
            assert f"ctas_per_tile={per_tile} " in plan
        check_forward(w, y_tol=1e-2)
        y1, i1, w1 = run_forward(w)
        y2, i2, w2 = run_forward(w)
        np.testing.assert_array_equal(y1, y2)                        # fixed summation order: reproducible bit for bit
        np.testing.assert_array_equal(i1, i2)
        np.testing.assert_array_equal(w1, w2)
    finally:
        mb.meteora_set_tuning("splits", 0)


# Adapter counts and ranks that change the stacked shrink's tiles (Wg behind A's rows, in a tile of its own, three
# tiles of A, nine with 128 adapters) and the width of the staged B rows.
@pytest.mark.parametrize("N,k,T,r", [(4, 2, 9, 8), (16, 4, 40, 8), (33, 3, 128, 8), (2, 1, 3, 8), (28, 2, 20, 16),
                                     (28, 2, 128, 32), (10, 3, 64, 24), (128, 2, 64, 8), (100, 8, 7, 8),
                                     (72, 4, 128, 16), (28, 1, 128, 8), (28, 2, 33, 8)])
def test_streamed_decode_kernel_adapter_counts(N, k, T, r):
    w = workloads.make_workload("stream_n", T=T, d_in=768, d_out=896, N=N, k=k, r=r, dtype="bf16", x_kind="normal",
                                seed=1900 + N + r, b_std=0.3, temperature=1.0 if N != 16 else 15.0)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16, w.temperature)
    assert "stream_decode" in mb.meteora_describe_plan(shape)
    check_forward(w, y_tol=1e-2)


def test_streamed_decode_kernel_rank_64_takes_one_aux_cta_per_stacked_tile():
    # 28 adapters of rank 64: 15 tiles of stacked rows.  With four aux CTAs per tile only two main CTAs per row tile
    # remain and the B rows of all adapters for a CTA's 64 output rows (229 KB) do not fit; the planner falls back
    # to one aux CTA per stacked tile, four main CTAs per row tile and 114 KB of staged rows.
    for T in (32, 1, 64):                                            # (at 128 tokens the landing area no longer fits either)
        w = workloads.make_workload("stream_r64", T=T, d_in=512, d_out=4096, N=28, k=2, r=64, dtype="bf16",
                                    x_kind="normal", seed=2700 + T, b_std=0.3)
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        plan = mb.meteora_describe_plan(shape)
        assert "stream_decode" in plan and "aux_ctas=15 " in plan and "ctas_per_tile=4 " in plan, plan
        check_forward(w, y_tol=1e-2)


# Its planner's choices forced the other way: a shallow ring, two k-steps per stage, no L2 prefetch, a small prefetch
# cap, one CTA per SM with a deep ring, few and many aux CTAs, no programmatic dependent launch.  None of them may
# change the result beyond the order of the fp32 sums of the stacked shrink's slices.  (pair_decode = 1 runs the 70
# tokens on pairs of CTAs with a two-CTA MMA, own_local = 0 sends a CTA's own row slice through scratch too.)
@pytest.mark.parametrize("knob,value", [("stages", 2), ("kc", 2), ("pf", -1), ("pf", 1), ("stream", 2), ("aux_ctas", 4),
                                        ("aux_ctas", 40), ("pdl_decode", 0), ("pair_decode", 1), ("own_local", 0), ("bulk_deliver", 1),
                                        ("aux_plain", 0)])
def test_streamed_decode_kernel_planner_choices(knob, value):
    w = workloads.make_workload("stream_knobs", T=70, d_in=2048, d_out=640, dtype="bf16", x_kind="normal", seed=2234,
                                b_std=0.3)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    y0, i0, _ = run_forward(w)
    default = {"stream": 1, "pdl_decode": 1, "own_local": 1, "aux_plain": 1}.get(knob, 0)
    mb.meteora_set_tuning(knob, value)
    try:
        assert "stream_decode" in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
        y1, i1, _ = run_forward(w)
    finally:
        mb.meteora_set_tuning(knob, default)
    same = assert_same_outside_the_band(w, i0, i1)
    assert same.mean() > 0.97
    assert rel_l2(y1[same], y0[same]) < 4e-3


@pytest.mark.parametrize("d_in,d_out,T,per_tile", [(1024, 640, 20, 0), (1024, 896, 33, 2), (2048, 4224, 48, 0)])
def test_streamed_decode_kernel_on_pairs_at_small_batches(d_in, d_out, T, per_tile):
    # pairs of CTAs (two-CTA MMA, each CTA half of the token tile; a knob, off by default), forced here for token
    # tiles of 32 and 64, an odd number of row tiles (7: the last pair's second CTA has no rows) and 33 tiles
    w = workloads.make_workload("stream_pairs", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="rms",
                                seed=250 + T + d_out, b_std=0.3)
    mb.meteora_set_tuning("pair_decode", 2)
    mb.meteora_set_tuning("splits", per_tile)
    try:
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        assert "pairs=1" in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
        y1, i1, _ = run_forward(w)
        y2, i2, _ = run_forward(w)
        np.testing.assert_array_equal(y1, y2)
    finally:
        mb.meteora_set_tuning("pair_decode", 0)
        mb.meteora_set_tuning("splits", 0)


def test_streamed_decode_calls_share_one_workspace_back_to_back():
    # Eight calls in a row on ONE workspace without any synchronisation: a call's CTAs are resident while the call
    # ahead still runs, but touch the workspace (counters, scratch) only after that call has completed.
    T, d_in, d_out = 96, 1024, 768
    ws_list = [workloads.make_workload(f"shared_ws{i}", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="normal",
                                       seed=7100 + i, b_std=0.3) for i in range(8)]
    shape = mb.make_shape(T, d_in, d_out, 28, 8, 2, torch.bfloat16)
    assert "stream_decode" in mb.meteora_describe_plan(shape)
    dev = [to_dev(w, "x", "W0", "A", "B", "Wg") for w in ws_list]
    workspace = mb.alloc_workspace(shape)
    ys = [mb.meteora_linear_forward(*t, 2, workspace=workspace) for t in dev]
    torch.cuda.synchronize()
    assert mb.meteora_workspace_status(workspace) == 0
    for w, t, y in zip(ws_list, dev, ys):
        y_alone, idx, _ = mb.meteora_linear_forward(*t, 2, return_routing=True)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(y.float().cpu().numpy(), y_alone.float().cpu().numpy())
        ref = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx.cpu().numpy())
        assert rel_l2(y.float().cpu().numpy(), ref) <= 1e-2


# --------------------------------------------------------------------------------------- clustered decode kernel
# The decode kernel whose CTAs of a row tile form a thread-block cluster and exchange through distributed shared
# memory, with the stacked shrink spread over all CTAs.  Shapes for every way its work splits: clusters of 1, 2, 3,
# 4, 5, 7 and 8 (even and uneven row slices), k-steps that do not divide by the cluster size (17), fewer k-steps per
# CTA than clusters per stacked tile (512: 8 k-steps), more clusters than stacked slices are used (71 row tiles),
# a ragged last tile (1000, 1001 rows), one token, a token count that is no multiple of 16, the full 128, more
# tokens than CTAs (128 tokens on 10 x 2 CTAs: several tokens per selecting CTA).
@pytest.fixture
def clustered_decode_kernel():
    mb.meteora_set_tuning("cluster_decode", 2)
    mb.meteora_set_tuning("wait_limit_us", 200000)                   # a wait that cannot end gives up after 0.2 s
    yield
    mb.meteora_set_tuning("wait_limit_us", 0)
    mb.meteora_set_tuning("cluster_decode", CLUSTER_DEFAULT)


CLUSTER_DEFAULT = 0


@pytest.mark.parametrize("d_in,d_out,T,per_tile", [
    (1024, 640, 1, 0), (1024, 640, 8, 0), (1024, 640, 100, 0), (1024, 640, 128, 0),
    (1536, 1000, 37, 0), (1088, 768, 16, 0), (2048, 4224, 5, 0), (2048, 4224, 128, 0),
    (512, 9000, 24, 0), (1024, 1280, 64, 1), (1024, 1280, 128, 2), (1024, 1280, 77, 3), (1024, 1001, 50, 5),
    (1024, 384, 128, 7), (1024, 384, 19, 8), (4096, 1024, 128, 0), (4096, 4096, 128, 0), (4096, 4096, 1, 0),
])
def test_clustered_decode_kernel_matches_oracle(d_in, d_out, T, per_tile, clustered_decode_kernel):
    w = workloads.make_workload("cluster", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="rms",
                                seed=350 + T + d_out, b_std=0.3)
    mb.meteora_set_tuning("splits", per_tile)
    try:
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        plan = mb.meteora_describe_plan(shape)
        assert "cluster_decode" in plan
        if per_tile:
            assert f"cluster={per_tile} " in plan
        check_forward(w, y_tol=1e-2)
        y1, i1, w1 = run_forward(w)
        y2, i2, w2 = run_forward(w)
        np.testing.assert_array_equal(y1, y2)                        # fixed summation order: reproducible bit for bit
        np.testing.assert_array_equal(i1, i2)
        np.testing.assert_array_equal(w1, w2)
    finally:
        mb.meteora_set_tuning("splits", 0)


@pytest.mark.parametrize("N,k,T,r", [(4, 2, 9, 8), (16, 4, 40, 8), (33, 3, 128, 8), (2, 1, 3, 8), (28, 2, 20, 16),
                                     (12, 2, 128, 32), (10, 3, 64, 24), (64, 8, 7, 8), (28, 1, 128, 8), (28, 2, 33, 8)])
def test_clustered_decode_kernel_adapter_counts(N, k, T, r, clustered_decode_kernel):
    w = workloads.make_workload("cluster_n", T=T, d_in=768, d_out=896, N=N, k=k, r=r, dtype="bf16", x_kind="normal",
                                seed=2900 + N + r, b_std=0.3, temperature=1.0 if N != 16 else 15.0)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16, w.temperature)
    assert "cluster_decode" in mb.meteora_describe_plan(shape)
    check_forward(w, y_tol=1e-2)


@pytest.mark.parametrize("knob,value", [("stages", 2), ("pdl_decode", 0), ("splits", 2)])
def test_clustered_decode_kernel_planner_choices(knob, value, clustered_decode_kernel):
    w = workloads.make_workload("cluster_knobs", T=70, d_in=2048, d_out=640, dtype="bf16", x_kind="normal", seed=3234,
                                b_std=0.3)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    y0, i0, _ = run_forward(w)
    mb.meteora_set_tuning(knob, value)
    try:
        assert "cluster_decode" in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
        y1, i1, _ = run_forward(w)
    finally:
        mb.meteora_set_tuning(knob, {"pdl_decode": 1}.get(knob, 0))
    same = assert_same_outside_the_band(w, i0, i1)
    assert same.mean() > 0.97
    assert rel_l2(y1[same], y0[same]) < 4e-3


def test_clustered_decode_calls_share_one_workspace_back_to_back(clustered_decode_kernel):
    T, d_in, d_out = 96, 1024, 768
    ws_list = [workloads.make_workload(f"shared_cl{i}", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="normal",
                                       seed=8100 + i, b_std=0.3) for i in range(8)]
    shape = mb.make_shape(T, d_in, d_out, 28, 8, 2, torch.bfloat16)
    assert "cluster_decode" in mb.meteora_describe_plan(shape)
    dev = [to_dev(w, "x", "W0", "A", "B", "Wg") for w in ws_list]
    workspace = mb.alloc_workspace(shape)
    ys = [mb.meteora_linear_forward(*t, 2, workspace=workspace) for t in dev]
    torch.cuda.synchronize()
    assert mb.meteora_workspace_status(workspace) == 0
    for w, t, y in zip(ws_list, dev, ys):
        y_alone, idx, _ = mb.meteora_linear_forward(*t, 2, return_routing=True)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(y.float().cpu().numpy(), y_alone.float().cpu().numpy())
        ref = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx.cpu().numpy())
        assert rel_l2(y.float().cpu().numpy(), ref) <= 1e-2


def test_a_nearly_empty_last_wave_of_pair_tiles_runs_as_small_tiles():
    # 8 row pairs x 10 token tiles = 80 pair tiles on 74 pairs of SMs: the planner carves the 6 tiles of the second
    # wave (last token tile of the last 6 row pairs) out of the pair launch; a launch of 128 x 64 tiles follows.
    # Forced to other sizes as well (1 row pair, all 8), with a ragged last token tile and rank 16.
    for T, r, carve in ((2560, 8, 0), (2500, 8, 1), (2500, 16, 8), (700, 8, 3)):
        w = workloads.make_workload("carve", T=T, d_in=512, d_out=2048, N=28, k=2, r=r, dtype="bf16", x_kind="normal",
                                    seed=9100 + T + carve, b_std=0.3)
        mb.meteora_set_tuning("pair", 2)
        mb.meteora_set_tuning("tail_carve", carve)
        try:
            shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
            plan = mb.meteora_describe_plan(shape)
            assert "pairs_of_ctas" in plan
            want = carve if carve else 6
            assert f"tail_pairs_as_small_tiles={want}" in plan, plan
            check_forward(w, y_tol=1e-2)
            y1, i1, _ = run_forward(w)
            mb.meteora_set_tuning("tail_carve", -1)                      # the same call with every tile on pairs
            assert "tail_pairs_as_small_tiles=0" in mb.meteora_describe_plan(shape)
            y0, i0, _ = run_forward(w)
            np.testing.assert_array_equal(i0, i1)
            assert rel_l2(y1, y0) < 2e-3
        finally:
            mb.meteora_set_tuning("pair", 1)
            mb.meteora_set_tuning("tail_carve", 0)


# Prefill base product on pairs of SMs (256 x 256 tiles): an odd number of row tiles (640 = 5, the last pair has
# one idle half), a ragged last token tile, a token count that leaves the second half of a pair's tokens empty
# (257), a contraction length that is no multiple of 64, and adapters up to an odd count.  The stacked shrink of
# these calls runs on pairs as well: its rows are [A; Wg] packed into 128-row tiles, two tiles per pair.
@pytest.mark.parametrize("d_in,d_out,T,N,k,r", [
    (1024, 640, 600, 28, 2, 8), (512, 256, 257, 28, 2, 8), (1096, 512, 300, 28, 2, 8), (768, 1024, 1024, 7, 3, 8),
    (512, 512, 520, 16, 4, 8), (512, 384, 300, 33, 3, 8),      # Wg in a tile of its own; three tiles of stacked rows
    (512, 384, 700, 28, 2, 16), (512, 256, 300, 28, 4, 64), (512, 256, 520, 5, 2, 24),   # ranks 16, 64, 24: 2, 8, 1 rounds
    (512, 512, 600, 128, 2, 8), (768, 256, 1100, 100, 4, 8),   # 128 and 100 adapters: 5 and 4 rounds of expand columns
])
def test_prefill_on_pairs_of_sms_matches_oracle(d_in, d_out, T, N, k, r):
    w = workloads.make_workload("pairs", T=T, d_in=d_in, d_out=d_out, N=N, k=k, r=r, dtype="bf16", x_kind="normal",
                                seed=700 + T, b_std=0.3)
    mb.meteora_set_tuning("pair", 2)                                 # 2: also where only a few pairs result
    try:
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        assert "pairs_of_ctas" in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
        y1, i1, _ = run_forward(w)
        y2, i2, _ = run_forward(w)
        np.testing.assert_array_equal(y1, y2)
    finally:
        mb.meteora_set_tuning("pair", 1)


def test_pairs_of_sms_over_several_waves():
    # 10 row pairs x 19 token tiles = 190 pair tiles on 74 pairs of SMs: three waves, the last token tile ragged.
    # y is compared on sampled tokens of every token tile (the oracle takes the GPU's own routing there).
    w = workloads.make_workload("pairs_waves", T=4700, d_in=512, d_out=2560, dtype="bf16", x_kind="normal",
                                seed=4700, b_std=0.3)
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    assert "pairs_of_ctas" in mb.meteora_describe_plan(shape)
    rng = np.random.default_rng(5)
    tokens = np.unique(np.concatenate([np.arange(0, w.T, 256), np.arange(127, w.T, 256), np.arange(128, w.T, 256),
                                       np.array([w.T - 1]), rng.integers(0, w.T, 200)]))
    check_forward(w, y_tol=1e-2, tokens=tokens)


@pytest.mark.parametrize("d_in,d_out,T", [(1024, 640, 600), (1096, 512, 300)])
def test_prefill_on_single_sms_matches_oracle(d_in, d_out, T):
    # the 128 x 256 tiles of one CTA each, which small prefill problems still take by default
    w = workloads.make_workload("single", T=T, d_in=d_in, d_out=d_out, dtype="bf16", x_kind="normal",
                                seed=800 + T, b_std=0.3)
    mb.meteora_set_tuning("pair", 0)
    try:
        shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
        assert "pairs_of_ctas" not in mb.meteora_describe_plan(shape)
        check_forward(w, y_tol=1e-2)
    finally:
        mb.meteora_set_tuning("pair", 1)


def test_chain_and_single_launch_paths_agree():
    w = workloads.config1(128)
    y_f, i_f, _ = run_forward(w)                                     # T = 128 takes a single launch by default
    mb.meteora_set_tuning("fused", 0)
    try:
        y_c, i_c, _ = run_forward(w)
    finally:
        mb.meteora_set_tuning("fused", 1)
    same = assert_same_outside_the_band(w, i_f, i_c)
    assert same.mean() > 0.98
    assert rel_l2(y_f[same], y_c[same]) < 5e-3


def test_host_buffer_entry_point():
    w = workloads.config1(8)
    _, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    x_host = torch.from_numpy(w["x"]).to(torch.bfloat16).pin_memory()
    y_host = torch.empty((w.T, w.d_out), dtype=torch.bfloat16).pin_memory()
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.bfloat16)
    ws = mb.alloc_workspace(shape)
    mb.meteora_linear_forward_host(x_host, W0, A, B, Wg, w.k, y_host, ws)
    assert mb.meteora_workspace_status(ws) == 0                      # synchronises
    y_dev, _, _ = run_forward(w)
    np.testing.assert_array_equal(y_host.float().numpy(), y_dev)


# ----------------------------------------------------------------------------------------- full-size shapes
# Every (shape, T) cell of configs 2, 3 and 4 at full size: the routing of all T tokens against the oracle, y on
# sampled tokens (first, last, the edges of the 128- and 256-token tiles, and random ones), all d_out outputs of each.
def sampled_tokens(T, seed, n=18):
    edges = [t for t in (0, 127, 128, 255, 256, T // 2, T - 257, T - 129, T - 1) if 0 <= t < T]
    return np.unique(np.concatenate([edges, np.random.default_rng(seed).integers(0, T, min(n, T))]).astype(np.int64))


@pytest.mark.parametrize("T", workloads.CONFIG2_T)
@pytest.mark.parametrize("shape", list(workloads.CONFIG2_SHAPES))
def test_config2_prefill_sampled_rows(shape, T):
    w = workloads.config2(shape, T)
    check_forward(w, y_tol=1e-2, tokens=sampled_tokens(T, 5))


@pytest.mark.parametrize("T", workloads.CONFIG3_T)
@pytest.mark.parametrize("shape", list(workloads.CONFIG3_SHAPES))
def test_config3_sampled_rows(shape, T):
    w = workloads.config3(shape, T)
    check_forward(w, y_tol=1e-2, tokens=sampled_tokens(T, 6))


@pytest.mark.parametrize("T", workloads.CONFIG4_T)
@pytest.mark.parametrize("linear", list(workloads.CONFIG4_LINEARS))
def test_config4_linears(linear, T):
    w = workloads.config4(linear, T)
    check_forward(w, y_tol=1e-2, tokens=sampled_tokens(T, 7))


# ----------------------------------------------------------------------------------------- error behaviour
def test_errors_are_reported_not_launched():
    w = workloads.config0()
    x, W0, A, B, Wg = to_dev(w, "x", "W0", "A", "B", "Wg")
    small = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(mb.MeteoraError) as e:
        mb.meteora_linear_forward(x, W0, A, B, Wg, 2, workspace=small)
    assert e.value.status == -4
    with pytest.raises(mb.MeteoraError) as e:
        mb.meteora_gate_topk(x, Wg, 5)
    assert e.value.status == -1
    with pytest.raises(mb.MeteoraError) as e:
        mb.meteora_linear_forward(x, W0, A, B, Wg, 2, temperature=0.0)
    assert e.value.status == -1
    shape = mb.make_shape(w.T, w.d_in, w.d_out, w.N, w.r, w.k, torch.float32)
    ws = mb.alloc_workspace(shape)
    lib = mb.load_library()
    import ctypes
    rc = lib.meteora_linear_forward(x.data_ptr() + 4, W0.data_ptr(), A.data_ptr(), B.data_ptr(), Wg.data_ptr(),
                                    ctypes.byref(shape), torch.empty_like(x).data_ptr(), ws.data_ptr(), ws.numel(),
                                    None)
    assert rc == -3
    y = mb.meteora_linear_forward(x[:0].contiguous(), W0, A, B, Wg, 2)   # T = 0 is a no-op
    assert y.shape == (0, w.d_out)
