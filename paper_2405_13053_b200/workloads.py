"""Seeded synthetic workloads for a MeteoRA linear layer.

This module only draws random tensors; it holds none of the method's
arithmetic.  Both the GPU tests/benchmark and the CPU oracle consume its
output, so the two sides see the same bytes.

Tensors follow the layer's storage convention (row-major, contiguous):
    x[T,d_in]  W0[d_out,d_in]  A[N,r,d_in]  B[N,d_out,r]  Wg[N,d_in]

Distributions (second argument of N(.,.) is the standard deviation):
    W0 ~ N(0, 0.02)     A_i ~ U(-1/sqrt(d_in), 1/sqrt(d_in))
    B_i ~ N(0, b_std)   (b_std = 0.01 unless stated)
    Wg ~ N(0, 1/sqrt(d_in))
    x  : "normal"   N(0,1)
         "rms"      N(0,1), then every token divided by its root mean square
         "clusters" 4 cluster means mu_c ~ N(0,1)^d_in; tokens come in 4
                    contiguous runs of T/4, x = mu_c + N(0,0.5)
They stand in for the paper's efficiency workloads (random pseudo data swept
over batch, sequence, top-k, rank, adapters and hidden sizes, App. A.7) at
LLaMA3-8B / LLaMA2-13B projection shapes with 28 adapters of rank 8, top-2.

Every tensor has its own PCG64 stream seeded by (seed, tensor number), so a
tensor does not change when another one is resized.  For "bf16" workloads each
tensor is rounded to bfloat16 (round-to-nearest-even) once, here, and handed
out as float32 holding exactly those values.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict

import numpy as np

_TENSOR_ID = {"x": 0, "W0": 1, "A": 2, "B": 3, "Wg": 4, "mu": 5}


def _rng(seed: int, name: str) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), _TENSOR_ID[name]])))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result is float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


@dataclasses.dataclass
class Workload:
    name: str
    T: int
    d_in: int
    d_out: int
    N: int
    r: int
    k: int
    dtype: str            # "f32" or "bf16": storage type of x, W0, A, B, Wg and y
    temperature: float
    seed: int
    x_kind: str
    tensors: Dict[str, np.ndarray]

    def __getitem__(self, key: str) -> np.ndarray:
        return self.tensors[key]


def make_x(T: int, d_in: int, x_kind: str, seed: int, dtype: str) -> np.ndarray:
    g = _rng(seed, "x")
    if x_kind == "normal":
        x = g.standard_normal((T, d_in), dtype=np.float32)
    elif x_kind == "rms":
        x = g.standard_normal((T, d_in), dtype=np.float32)
        rms = np.sqrt(np.mean(x.astype(np.float64) ** 2, axis=1, keepdims=True))
        x = (x / np.maximum(rms, 1e-12)).astype(np.float32)
    elif x_kind == "clusters":
        mu = _rng(seed, "mu").standard_normal((4, d_in), dtype=np.float32)
        x = np.float32(0.5) * g.standard_normal((T, d_in), dtype=np.float32)
        run = -(-T // 4) if T > 0 else 1
        cluster = np.minimum(np.arange(T) // max(run, 1), 3)
        x += mu[cluster]
    else:
        raise ValueError(f"unknown x_kind {x_kind!r}")
    return round_to_bf16(x) if dtype == "bf16" else x


def make_workload(name: str, T: int, d_in: int, d_out: int, N: int = 28, r: int = 8, k: int = 2,
                  dtype: str = "bf16", x_kind: str = "normal", seed: int = 0, b_std: float = 0.01,
                  temperature: float = 1.0) -> Workload:
    if dtype not in ("f32", "bf16"):
        raise ValueError("dtype must be 'f32' or 'bf16'")
    fin = 1.0 / math.sqrt(d_in)
    t: Dict[str, np.ndarray] = {}
    t["x"] = make_x(T, d_in, x_kind, seed, dtype)
    t["W0"] = np.float32(0.02) * _rng(seed, "W0").standard_normal((d_out, d_in), dtype=np.float32)
    t["A"] = _rng(seed, "A").uniform(-fin, fin, size=(N, r, d_in)).astype(np.float32)
    t["B"] = np.float32(b_std) * _rng(seed, "B").standard_normal((N, d_out, r), dtype=np.float32)
    t["Wg"] = np.float32(fin) * _rng(seed, "Wg").standard_normal((N, d_in), dtype=np.float32)
    if dtype == "bf16":
        for key in ("W0", "A", "B", "Wg"):
            t[key] = round_to_bf16(t[key])
    return Workload(name, T, d_in, d_out, N, r, k, dtype, float(temperature), int(seed), x_kind, t)


# ---------------------------------------------------------------------------------------------
# The named configurations.  seed = 1000 * config + index of the (shape, T) pair in the config.
# ---------------------------------------------------------------------------------------------
CONFIG1_T = (1, 8, 32, 128)
CONFIG2_SHAPES = {"gate_up": (4096, 14336), "down": (14336, 4096), "kv": (4096, 1024)}
CONFIG2_T = (512, 2048, 8192)
CONFIG3_SHAPES = {"qkvo": (5120, 5120), "gate_up": (5120, 13824), "down": (13824, 5120)}
CONFIG3_T = (1, 64, 4096)
CONFIG4_LINEARS = {"q": (4096, 4096), "k": (4096, 1024), "v": (4096, 1024), "o": (4096, 4096),
                   "gate": (4096, 14336), "up": (4096, 14336), "down": (14336, 4096)}
CONFIG4_T = (64, 4096)


def config0(**kw) -> Workload:
    """Tiny fp32 correctness case: 256 -> 256, 4 adapters, rank 8, top-2, 64 tokens, seed 0."""
    return make_workload("config0", T=64, d_in=256, d_out=256, N=4, r=8, k=2, dtype="f32",
                         x_kind="normal", seed=0, **kw)


def config1(T: int, **kw) -> Workload:
    """LLaMA3-8B q_proj shape, decode batch: 4096 -> 4096, RMS-normalised tokens."""
    index = CONFIG1_T.index(T) if T in CONFIG1_T else 100 + T
    return make_workload(f"config1/T{T}", T=T, d_in=4096, d_out=4096, x_kind="rms",
                         seed=1000 + index, **kw)


def config2(shape: str, T: int, **kw) -> Workload:
    """LLaMA3-8B MLP and k/v shapes, prefill, tokens from 4 clusters (skewed routing)."""
    d_in, d_out = CONFIG2_SHAPES[shape]
    si = list(CONFIG2_SHAPES).index(shape)
    ti = CONFIG2_T.index(T) if T in CONFIG2_T else 100 + T
    return make_workload(f"config2/{shape}/T{T}", T=T, d_in=d_in, d_out=d_out, x_kind="clusters",
                         seed=2000 + si * 10 + ti if ti < 10 else 2000 + si * 10000 + ti, **kw)


def config3(shape: str, T: int, **kw) -> Workload:
    """LLaMA2-13B shapes, x ~ N(0,1)."""
    d_in, d_out = CONFIG3_SHAPES[shape]
    si = list(CONFIG3_SHAPES).index(shape)
    ti = CONFIG3_T.index(T) if T in CONFIG3_T else 100 + T
    return make_workload(f"config3/{shape}/T{T}", T=T, d_in=d_in, d_out=d_out, x_kind="normal",
                         seed=3000 + si * 10 + ti if ti < 10 else 3000 + si * 10000 + ti, **kw)


def config4(linear: str, T: int, **kw) -> Workload:
    """One of the 7 MeteoRA linears of a LLaMA3-8B decoder layer, each with its own gate."""
    d_in, d_out = CONFIG4_LINEARS[linear]
    li = list(CONFIG4_LINEARS).index(linear)
    ti = CONFIG4_T.index(T) if T in CONFIG4_T else 100 + T
    return make_workload(f"config4/{linear}/T{T}", T=T, d_in=d_in, d_out=d_out, x_kind="rms",
                         seed=4000 + li * 10 + ti if ti < 10 else 4000 + li * 10000 + ti, **kw)
