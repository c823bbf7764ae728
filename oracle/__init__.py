"""CPU oracle for the MeteoRA linear forward.  TEST INFRASTRUCTURE ONLY.

`meteora_oracle.c` is the plain fp64 definition (Eq. 1-3 and Sec. 3.3 of the
MeteoRA paper); this package compiles it with gcc and exposes it through
ctypes.  Nothing here shares code with the CUDA library, and only the tests,
the smoke check and the benchmark's CPU legs may import it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "meteora_oracle.c")
_LIB = os.path.join(_HERE, "libmeteora_oracle.so")
_lock = threading.Lock()
_lib = None

_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
                   "-o", _LIB, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c_int, c_double = ctypes.c_int, ctypes.c_double
        lib.meteora_oracle_num_threads.restype = c_int
        lib.meteora_oracle_set_threads.argtypes = [c_int]
        lib.meteora_oracle_set_threads.restype = None
        lib.meteora_oracle_gate_topk.argtypes = [_f32p, _f32p, c_int, c_int, c_int, c_int, c_double,
                                                 _i32p, _f64p, _f32p]
        lib.meteora_oracle_route.argtypes = [_i32p, c_int, c_int, c_int, _i32p, _i32p, _i32p]
        lib.meteora_oracle_lora_delta.argtypes = [_f32p, _f32p, _f32p, _i32p, _f32p] + [c_int] * 6 + [_f64p]
        lib.meteora_oracle_linear_forward.argtypes = [_f32p] * 5 + [c_int] * 6 + [c_double, _f64p, _i32p, _f64p]
        lib.meteora_oracle_linear_forward_routed.argtypes = [_f32p] * 5 + [_i32p] + [c_int] * 6 + [c_double, _f64p]
        lib.meteora_oracle_gate_backward.argtypes = [_f32p] * 5 + [_i32p] + [c_int] * 6 + [c_double, _f64p, _f64p]
        _lib = lib
    return _lib


def _f32(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _i32(a, shape):
    a = np.ascontiguousarray(a, dtype=np.int32)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _p(a, ty):
    return a.ctypes.data_as(ty)


def _check(status: int, what: str):
    if status != 0:
        raise ValueError(f"oracle {what}: invalid argument (status {status})")


def num_threads() -> int:
    return int(_load().meteora_oracle_num_threads())


def set_threads(n: int) -> None:
    _load().meteora_oracle_set_threads(int(n))


def gate_topk(x, Wg, k, temperature=1.0):
    """Sec. 3.1 + Eq. 3. Returns (topk_idx[T,k] int32, topk_w[T,k] float64, logits[T,N] float32)."""
    T, d_in = x.shape
    N = Wg.shape[0]
    x, Wg = _f32(x, (T, d_in)), _f32(Wg, (N, d_in))
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    logits = np.empty((T, N), np.float32)
    _check(_load().meteora_oracle_gate_topk(_p(x, _f32p), _p(Wg, _f32p), T, d_in, N, k, float(temperature),
                                            _p(idx, _i32p), _p(w, _f64p), _p(logits, _f32p)), "gate_topk")
    return idx, w, logits


def route(topk_idx, N):
    """Sec. 3.3 grouping. Returns (counts[N], offsets[N+1], perm[T*k]) int32."""
    T, k = topk_idx.shape
    idx = _i32(topk_idx, (T, k))
    counts = np.empty(N, np.int32)
    offsets = np.empty(N + 1, np.int32)
    perm = np.empty(T * k, np.int32)
    _check(_load().meteora_oracle_route(_p(idx, _i32p), T, k, N, _p(counts, _i32p), _p(offsets, _i32p),
                                        _p(perm, _i32p)), "route")
    return counts, offsets, perm


def lora_delta(x, A, B, topk_idx, topk_w):
    """LoRA term of Eq. 2 for given routing. Returns delta[T,d_out] float64."""
    T, d_in = x.shape
    N, r, _ = A.shape
    d_out = B.shape[1]
    k = topk_idx.shape[1]
    x, A, B = _f32(x, (T, d_in)), _f32(A, (N, r, d_in)), _f32(B, (N, d_out, r))
    idx, w = _i32(topk_idx, (T, k)), _f32(topk_w, (T, k))
    delta = np.empty((T, d_out), np.float64)
    _check(_load().meteora_oracle_lora_delta(_p(x, _f32p), _p(A, _f32p), _p(B, _f32p), _p(idx, _i32p),
                                             _p(w, _f32p), T, d_in, d_out, N, r, k, _p(delta, _f64p)),
           "lora_delta")
    return delta


def linear_forward(x, W0, A, B, Wg, k, temperature=1.0):
    """Eq. 2 + Eq. 3. Returns (y[T,d_out] float64, topk_idx[T,k] int32, topk_w[T,k] float64)."""
    T, d_in = x.shape
    d_out = W0.shape[0]
    N, r, _ = A.shape
    x, W0 = _f32(x, (T, d_in)), _f32(W0, (d_out, d_in))
    A, B, Wg = _f32(A, (N, r, d_in)), _f32(B, (N, d_out, r)), _f32(Wg, (N, d_in))
    y = np.empty((T, d_out), np.float64)
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    _check(_load().meteora_oracle_linear_forward(_p(x, _f32p), _p(W0, _f32p), _p(A, _f32p), _p(B, _f32p),
                                                 _p(Wg, _f32p), T, d_in, d_out, N, r, k, float(temperature),
                                                 _p(y, _f64p), _p(idx, _i32p), _p(w, _f64p)), "linear_forward")
    return y, idx, w


def linear_forward_routed(x, W0, A, B, Wg, topk_idx, temperature=1.0):
    """Eq. 2 with a given selection (weights by Eq. 3 on this side's logits). Returns y float64."""
    T, d_in = x.shape
    d_out = W0.shape[0]
    N, r, _ = A.shape
    k = topk_idx.shape[1]
    x, W0 = _f32(x, (T, d_in)), _f32(W0, (d_out, d_in))
    A, B, Wg = _f32(A, (N, r, d_in)), _f32(B, (N, d_out, r)), _f32(Wg, (N, d_in))
    idx = _i32(topk_idx, (T, k))
    y = np.empty((T, d_out), np.float64)
    _check(_load().meteora_oracle_linear_forward_routed(_p(x, _f32p), _p(W0, _f32p), _p(A, _f32p),
                                                        _p(B, _f32p), _p(Wg, _f32p), _p(idx, _i32p), T, d_in,
                                                        d_out, N, r, k, float(temperature), _p(y, _f64p)),
           "linear_forward_routed")
    return y


def gate_backward(x, A, B, Wg, dy, topk_idx, temperature=1.0):
    """Gradient of the gate weights through Eq. 3 and Eq. 2 for a given selection (Sec. 3.2).
    Returns (dlogit[T,k] float64, dWg[N,d_in] float64)."""
    T, d_in = x.shape
    N, r, _ = A.shape
    d_out = B.shape[1]
    k = topk_idx.shape[1]
    x, A, B = _f32(x, (T, d_in)), _f32(A, (N, r, d_in)), _f32(B, (N, d_out, r))
    Wg, dy, idx = _f32(Wg, (N, d_in)), _f32(dy, (T, d_out)), _i32(topk_idx, (T, k))
    dlogit = np.empty((T, k), np.float64)
    dWg = np.empty((N, d_in), np.float64)
    _check(_load().meteora_oracle_gate_backward(_p(x, _f32p), _p(A, _f32p), _p(B, _f32p), _p(Wg, _f32p),
                                                _p(dy, _f32p), _p(idx, _i32p), T, d_in, d_out, N, r, k,
                                                float(temperature), _p(dlogit, _f64p), _p(dWg, _f64p)),
           "gate_backward")
    return dlogit, dWg
