"""Pins for the CPU oracle: every check compares it with something that is not the oracle.

The references used here are the paper's definitions worked out by hand
(tests/golden), closed forms, invariants of Eq. 2 / Eq. 3, and special cases that
reduce to numpy / scipy library routines (matrix product, stable argsort, softmax).
Shapes are deliberately non-square (d_in != d_out, r != k != N) so that a transposed
operand or a swapped index cannot pass.
"""
import math

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

import oracle
from paper_2405_13053_b200 import workloads


def small(seed=7, T=13, d_in=24, d_out=20, N=5, r=3, k=2, b_std=0.3, dtype="f32"):
    return workloads.make_workload("pin", T=T, d_in=d_in, d_out=d_out, N=N, r=r, k=k, dtype=dtype,
                                   x_kind="normal", seed=seed, b_std=b_std)


def f64(a):
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------- Eq. 2, base term
def test_zero_B_gives_plain_matrix_product():
    w = small()
    y, _, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], np.zeros_like(w["B"]), w["Wg"], w.k)
    np.testing.assert_allclose(y, f64(w["x"]) @ f64(w["W0"]).T, rtol=1e-13, atol=1e-13)


# --------------------------------------------------------------------------- Eq. 1 / App. A.1
@pytest.mark.parametrize("forced", [0, 3, 4])
def test_top1_forced_gate_is_single_lora(forced):
    w = small(seed=11 + forced, k=1)
    x = w["x"].copy()
    x[:, 0] = 1.0                                   # a constant feature the gate can key on
    Wg = np.zeros_like(w["Wg"])
    Wg[forced, 0] = 50.0
    Wg[:, 1:] = 0.01 * w["Wg"][:, 1:]
    y, idx, wts = oracle.linear_forward(x, w["W0"], w["A"], w["B"], Wg, 1)
    assert np.all(idx == forced)
    assert np.all(wts == 1.0)                       # softmax over one element is exactly 1
    X = f64(x)
    expect = X @ f64(w["W0"]).T + (X @ f64(w["A"][forced]).T) @ f64(w["B"][forced]).T
    np.testing.assert_allclose(y, expect, rtol=1e-12, atol=1e-12)


# --------------------------------------------------------------------------- Eq. 3
def test_weights_sum_to_one_positive_and_ordered():
    w = small(T=200, N=9, k=4)
    idx, wts, logits = oracle.gate_topk(w["x"], w["Wg"], 4)
    np.testing.assert_allclose(wts.sum(axis=1), 1.0, atol=1e-14)
    assert np.all(wts > 0)
    assert np.all(np.diff(wts, axis=1) <= 0)        # picks listed by descending logit
    picked = np.take_along_axis(logits, idx.astype(np.int64), axis=1)
    assert np.all(np.diff(picked, axis=1) <= 0)
    rest = logits.copy()
    np.put_along_axis(rest, idx.astype(np.int64), -np.inf, axis=1)
    assert np.all(rest.max(axis=1) <= picked[:, -1])  # nothing left out beats a selected logit


def test_two_logit_closed_form():
    # k = 2: w_0 = 1 / (1 + exp(-(l_0 - l_1))) -- the logistic function of the logit gap.
    w = small(T=50, N=6, k=2)
    idx, wts, logits = oracle.gate_topk(w["x"], w["Wg"], 2)
    picked = f64(np.take_along_axis(logits, idx.astype(np.int64), axis=1))
    gap = picked[:, 0] - picked[:, 1]
    np.testing.assert_allclose(wts[:, 0], 1.0 / (1.0 + np.exp(-gap)), rtol=1e-13)


def test_logits_match_library_product():
    w = small(T=40, N=7)
    _, _, logits = oracle.gate_topk(w["x"], w["Wg"], 2)
    ref = (f64(w["x"]) @ f64(w["Wg"]).T).astype(np.float32)
    assert logits.shape == (40, 7)
    np.testing.assert_allclose(logits, ref, rtol=2e-7, atol=1e-7)


def test_equal_logits_equal_weights_and_lower_index_first():
    w = small(N=6, k=3)
    Wg = w["Wg"].copy()
    Wg[4] = Wg[1]                                   # adapters 1 and 4 always tie
    Wg[1] *= 0
    Wg[4] *= 0
    Wg[1, 0] = Wg[4, 0] = 100.0
    x = w["x"].copy()
    x[:, 0] = 1.0
    idx, wts, _ = oracle.gate_topk(x, Wg, 3)
    assert np.all(idx[:, 0] == 1) and np.all(idx[:, 1] == 4)
    np.testing.assert_array_equal(wts[:, 0], wts[:, 1])


def test_all_logits_equal_picks_first_k():
    x = np.ones((3, 8), np.float32)
    Wg = np.zeros((5, 8), np.float32)
    idx, wts, _ = oracle.gate_topk(x, Wg, 3)
    np.testing.assert_array_equal(idx, np.tile(np.arange(3, dtype=np.int32), (3, 1)))
    np.testing.assert_allclose(wts, 1.0 / 3.0, rtol=1e-15)


def test_temperature_limits_and_scaling():
    w = small(T=30, N=6, k=3)
    idx1, w1, logits = oracle.gate_topk(w["x"], w["Wg"], 3, temperature=1.0)
    idx_hot, w_hot, _ = oracle.gate_topk(w["x"], w["Wg"], 3, temperature=1e9)
    np.testing.assert_array_equal(idx1, idx_hot)     # temperature never changes the selection
    np.testing.assert_allclose(w_hot, 1.0 / 3.0, atol=1e-8)
    # dividing by tau equals the library softmax of the selected logits / tau
    tau = 15.0
    _, w_tau, _ = oracle.gate_topk(w["x"], w["Wg"], 3, temperature=tau)
    picked = f64(np.take_along_axis(logits, idx1.astype(np.int64), axis=1))
    np.testing.assert_allclose(w_tau, scipy_softmax(picked / tau, axis=1), rtol=1e-13)


# --------------------------------------------------------------------------- hand-worked example
def _handworked():
    L = math.log(2.0)
    x = np.array([[1, 0], [0, 1]], np.float32)
    W0 = np.array([[1, 2], [3, 4]], np.float32)
    Wg = np.array([[2 * L, 0], [L, 3 * L], [0, L]], np.float32)
    A = np.array([[[3, 1]], [[-6, 5]], [[2, 10]]], np.float32)
    B = np.array([[[1], [2]], [[-1], [3]], [[5], [0]]], np.float32)
    return x, W0, A, B, Wg


def test_handworked_example(golden):
    g = golden("handworked_eq2_eq3.txt")
    x, W0, A, B, Wg = _handworked()
    y, idx, wts = oracle.linear_forward(x, W0, A, B, Wg, 2)
    np.testing.assert_array_equal(idx.ravel(), np.array(g["topk_idx"], np.int32))
    np.testing.assert_allclose(wts.ravel(), np.array(g["topk_w_num"]) / np.array(g["topk_w_den"]), rtol=1e-6)
    np.testing.assert_allclose(y.ravel(), g["y"], rtol=1e-6)
    delta = oracle.lora_delta(x, A, B, idx, wts.astype(np.float32))
    np.testing.assert_allclose(delta, [[4, -2], [6, 12]], rtol=1e-6)


def test_handworked_example_with_temperature(golden):
    g = golden("handworked_eq2_eq3.txt")
    x, W0, A, B, Wg = _handworked()
    y, idx, wts = oracle.linear_forward(x, W0, A, B, Wg, 2, temperature=2.0)
    np.testing.assert_allclose(wts[1], np.array(g["tau2_topk_w_token1_num"]) / np.array(g["tau2_topk_w_token1_den"]),
                               rtol=1e-6)
    np.testing.assert_allclose(y[1], np.array(g["tau2_y_token1_num"]) / np.array(g["tau2_y_token1_den"]), rtol=1e-6)
    s2 = math.sqrt(2.0)
    np.testing.assert_allclose(wts[0], [s2 / (1 + s2), 1 / (1 + s2)], rtol=1e-6)


# --------------------------------------------------------------------------- set semantics
def test_relabelling_adapters_leaves_output_unchanged():
    w = small(T=31, N=7, k=3)
    y, idx, wts = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], 3)
    p = np.random.default_rng(3).permutation(7)      # new adapter j is old adapter p[j]
    y2, idx2, wts2 = oracle.linear_forward(w["x"], w["W0"], w["A"][p], w["B"][p], w["Wg"][p], 3)
    np.testing.assert_allclose(y2, y, rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(p[idx2], idx)      # indices map through the relabelling
    np.testing.assert_allclose(wts2, wts, rtol=1e-13)


# --------------------------------------------------------------------------- Eq. 5, batched view
def _dense_masked(w, k, tau=1.0):
    """All N adapters evaluated for every token, multiplied by a gate vector that is zero off the top-k."""
    X, W0, A, B, Wg = (f64(w[n]) for n in ("x", "W0", "A", "B", "Wg"))
    logits = (X @ Wg.T).astype(np.float32).astype(np.float64)
    order = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    gate = np.zeros_like(logits)
    np.put_along_axis(gate, order, scipy_softmax(np.take_along_axis(logits, order, axis=1) / tau, axis=1), axis=1)
    U = np.einsum("nrd,td->tnr", A, X)
    D = np.einsum("nor,tnr->tno", B, U)
    return X @ W0.T + np.einsum("tn,tno->to", gate, D), order


@pytest.mark.parametrize("N,k,r", [(4, 2, 3), (3, 1, 2), (5, 5, 1), (28, 2, 8)])
def test_sparse_equals_masked_dense(N, k, r):
    w = small(seed=100 + N, T=17, d_in=32, d_out=12, N=N, r=r, k=k)
    y, idx, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], k)
    ref, order = _dense_masked(w, k)
    np.testing.assert_array_equal(idx, order)
    np.testing.assert_allclose(y, ref, rtol=1e-11, atol=1e-12)


def test_k_equals_N_is_full_softmax_mixture():
    w = small(T=9, N=4, k=4)
    y, _, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], 4)
    X, W0, A, B, Wg = (f64(w[n]) for n in ("x", "W0", "A", "B", "Wg"))
    gate = scipy_softmax((X @ Wg.T).astype(np.float32).astype(np.float64), axis=1)
    ref = X @ W0.T
    for n in range(4):
        ref += gate[:, n:n + 1] * ((X @ A[n].T) @ B[n].T)
    np.testing.assert_allclose(y, ref, rtol=1e-11, atol=1e-12)


# --------------------------------------------------------------------------- linearity
def test_top1_output_is_homogeneous_in_x():
    # k = 1: the weight is 1 whatever the scale, so y(a x) = a y(x) for a > 0.
    w = small(k=1)
    y1, idx1, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], 1)
    y4, idx4, _ = oracle.linear_forward(4.0 * w["x"], w["W0"], w["A"], w["B"], w["Wg"], 1)
    np.testing.assert_array_equal(idx1, idx4)
    np.testing.assert_allclose(y4, 4.0 * y1, rtol=1e-13)


def test_temperature_scaled_with_x_is_homogeneous():
    w = small(k=2)
    y1, _, w1 = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], 2, temperature=1.0)
    y2, _, w2 = oracle.linear_forward(2.0 * w["x"], w["W0"], w["A"], w["B"], w["Wg"], 2, temperature=2.0)
    np.testing.assert_allclose(w2, w1, rtol=1e-6)    # logits are rounded to float on both sides
    np.testing.assert_allclose(y2, 2.0 * y1, rtol=1e-6)


# --------------------------------------------------------------------------- LoRA term alone
def test_delta_is_forward_minus_base_and_matches_library():
    w = small(T=19, N=6, k=2, r=4)
    y, idx, wts = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], 2)
    y0, _, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], np.zeros_like(w["B"]), w["Wg"], 2)
    w32 = wts.astype(np.float32)
    delta = oracle.lora_delta(w["x"], w["A"], w["B"], idx, w32)
    np.testing.assert_allclose(delta, y - y0, rtol=1e-6, atol=1e-7)   # weights were rounded to float
    X, A, B = f64(w["x"]), f64(w["A"]), f64(w["B"])
    ref = np.zeros_like(delta)
    for t in range(w.T):
        for j in range(2):
            i = idx[t, j]
            ref[t] += float(w32[t, j]) * (B[i] @ (A[i] @ X[t]))
    np.testing.assert_allclose(delta, ref, rtol=1e-12, atol=1e-14)


def test_forward_routed_reproduces_forward_and_follows_given_selection():
    w = small(T=15, N=6, k=2)
    y, idx, _ = oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], 2)
    np.testing.assert_allclose(oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], idx), y,
                               rtol=1e-14)
    other = np.tile(np.array([[5, 0]], np.int32), (w.T, 1))
    y_other = oracle.linear_forward_routed(w["x"], w["W0"], w["A"], w["B"], w["Wg"], other)
    X, W0, A, B, Wg = (f64(w[n]) for n in ("x", "W0", "A", "B", "Wg"))
    lg = (X @ Wg.T).astype(np.float32).astype(np.float64)[:, [5, 0]]
    g = scipy_softmax(lg, axis=1)
    ref = X @ W0.T + g[:, :1] * ((X @ A[5].T) @ B[5].T) + g[:, 1:] * ((X @ A[0].T) @ B[0].T)
    np.testing.assert_allclose(y_other, ref, rtol=1e-11, atol=1e-12)


# --------------------------------------------------------------------------- routing (Sec. 3.3)
def test_route_handworked(golden):
    g = golden("handworked_route.txt")
    idx = np.array(g["topk_idx"], np.int32).reshape(3, 2)
    counts, offsets, perm = oracle.route(idx, 4)
    np.testing.assert_array_equal(counts, np.array(g["counts"], np.int32))
    np.testing.assert_array_equal(offsets, np.array(g["offsets"], np.int32))
    np.testing.assert_array_equal(perm, np.array(g["perm"], np.int32))


@pytest.mark.parametrize("T,k,N", [(1, 1, 1), (1, 2, 28), (37, 2, 28), (64, 3, 5), (500, 2, 28), (0, 2, 4)])
def test_route_equals_stable_argsort_and_invariants(T, k, N):
    rng = np.random.default_rng(T * 31 + k)
    idx = np.stack([rng.permutation(N)[:k] for _ in range(T)]).astype(np.int32) if T else np.zeros((0, k), np.int32)
    if T > 10:
        idx[: T // 2] = np.sort(rng.integers(0, min(N, 3), size=(T // 2, k)), axis=1)   # skew + empty adapters
    counts, offsets, perm = oracle.route(idx, N)
    flat = idx.ravel()
    np.testing.assert_array_equal(perm, np.argsort(flat, kind="stable").astype(np.int32))
    np.testing.assert_array_equal(counts, np.bincount(flat, minlength=N).astype(np.int32))
    assert counts.sum() == T * k and offsets[0] == 0 and offsets[-1] == T * k
    np.testing.assert_array_equal(np.diff(offsets), counts)
    assert sorted(perm.tolist()) == list(range(T * k))
    for e in range(N):
        seg = perm[offsets[e]:offsets[e + 1]]
        assert np.all(flat[seg] == e) and np.all(np.diff(seg) > 0)


# --------------------------------------------------------------------------- argument checks
def test_bad_arguments_are_rejected():
    w = small()
    with pytest.raises(ValueError):
        oracle.gate_topk(w["x"], w["Wg"], 0)
    with pytest.raises(ValueError):
        oracle.gate_topk(w["x"], w["Wg"], w.N + 1)
    with pytest.raises(ValueError):
        oracle.gate_topk(w["x"], w["Wg"], 2, temperature=0.0)
    with pytest.raises(ValueError):
        oracle.route(np.array([[0, 9]], np.int32), 4)


# --------------------------------------------------------------------------- bf16 workloads
def test_bf16_workload_values_are_exact_bf16():
    w = small(dtype="bf16")
    for name in ("x", "W0", "A", "B", "Wg"):
        bits = w[name].view(np.uint32)
        assert np.all((bits & 0xFFFF) == 0), name
    a = np.array([1.0, 1.00390625, 1.01171875, -3.0e-3], np.float32)   # 1+2^-8 ties to even -> 1.0
    np.testing.assert_array_equal(workloads.round_to_bf16(a)[:3], np.array([1.0, 1.0, 1.015625], np.float32))
