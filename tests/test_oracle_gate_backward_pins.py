"""Pins of the oracle's gate gradient (no GPU): a hand-worked case, central finite differences of the (already
pinned) routed forward with the selection held fixed, and the structure Eq. 3 imposes."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "handworked_gate_backward.txt")


def _golden():
    out = {}
    with open(GOLDEN) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def test_handworked_example():
    g = _golden()
    x = np.array([[1.0]], np.float32)
    Wg = np.array([[np.log(2.0)], [0.0]], np.float32)
    A = np.ones((2, 1, 1), np.float32)
    B = np.array([[[1.0]], [[4.0]]], np.float32)
    dy = np.array([[3.0]], np.float32)
    idx = np.array([[0, 1]], np.int32)
    dlogit, dWg = oracle.gate_backward(x, A, B, Wg, dy, idx)
    np.testing.assert_allclose(dlogit.ravel(), g["dlogit"], atol=1e-6)
    np.testing.assert_allclose(dWg.ravel(), g["dWg"], atol=1e-6)


def _case(seed, T=5, d_in=6, d_out=7, N=4, r=3, k=2):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, d_in)).astype(np.float32)
    W0 = rng.standard_normal((d_out, d_in)).astype(np.float32)
    A = rng.standard_normal((N, r, d_in)).astype(np.float32)
    B = rng.standard_normal((N, d_out, r)).astype(np.float32)
    Wg = rng.standard_normal((N, d_in)).astype(np.float32)
    c = rng.standard_normal((T, d_out)).astype(np.float32)          # L = sum c * y, so dL/dy = c
    return x, W0, A, B, Wg, c


def test_matches_finite_differences_of_the_forward():
    for tau in (1.0, 2.5):
        x, W0, A, B, Wg, c = _case(3)
        _, idx, _ = oracle.linear_forward(x, W0, A, B, Wg, 2, tau)
        _, dWg = oracle.gate_backward(x, A, B, Wg, c, idx, tau)
        h = 2.0 ** -7                                               # exactly representable steps
        num = np.zeros_like(dWg)
        for n in range(Wg.shape[0]):
            for d in range(Wg.shape[1]):
                Wp, Wm = Wg.copy(), Wg.copy()
                Wp[n, d] += h
                Wm[n, d] -= h
                Lp = float(np.sum(c * oracle.linear_forward_routed(x, W0, A, B, Wp, idx, tau)))
                Lm = float(np.sum(c * oracle.linear_forward_routed(x, W0, A, B, Wm, idx, tau)))
                num[n, d] = (Lp - Lm) / (2 * h)
        scale = np.abs(num).max()
        assert scale > 0.1
        np.testing.assert_allclose(dWg, num, atol=2e-3 * scale)     # O(h^2) truncation of the central difference


def test_top1_has_no_gradient_and_dlogits_sum_to_zero():
    x, W0, A, B, Wg, c = _case(4, k=1)
    _, idx1, _ = oracle.linear_forward(x, W0, A, B, Wg, 1)
    dlogit, dWg = oracle.gate_backward(x, A, B, Wg, c, idx1)
    assert np.all(dlogit == 0.0) and np.all(dWg == 0.0)              # App. A.1: the weight is the constant 1
    _, idx3, _ = oracle.linear_forward(x, W0, A, B, Wg, 3)
    dlogit, dWg = oracle.gate_backward(x, A, B, Wg, c, idx3)
    np.testing.assert_allclose(dlogit.sum(axis=1), 0.0, atol=1e-9)   # softmax: shifts of all logits change nothing
    untouched = np.setdiff1d(np.arange(Wg.shape[0]), np.unique(idx3))
    assert np.all(dWg[untouched] == 0.0)


def test_gradient_scales_with_inverse_temperature_at_equal_weights():
    # equal selected logits: w = 1/k for every temperature, so dlogit is exactly proportional to 1/tau
    x, W0, A, B, Wg, c = _case(5)
    Wg[:] = 0.0
    idx = np.tile(np.array([[1, 3]], np.int32), (x.shape[0], 1))
    d1, _ = oracle.gate_backward(x, A, B, Wg, c, idx, 1.0)
    d4, _ = oracle.gate_backward(x, A, B, Wg, c, idx, 4.0)
    np.testing.assert_allclose(d4, d1 / 4.0, rtol=1e-12, atol=1e-12)
