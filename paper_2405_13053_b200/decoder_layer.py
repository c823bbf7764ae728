"""A LLaMA3-8B decoder layer around the seven MeteoRA linears (Sec. 3.1: a MeteoRA module replaces each of q, k, v,
o, gate, up and down of every block; Sec. 3.2: every one of them has its own gate and adapters).

Only the seven linears are the library's; everything else (RMSNorm, rotary position embedding, grouped-query
attention with 32 query and 8 key/value heads of 128, SwiGLU, the two residual adds) runs as plain torch ops and
exists so that each linear consumes the real upstream activation:

    n1 = RMSNorm(x);  q, k, v = linears(n1);  rotary(q, k);  a = attention(q, [cache; k], [cache; v])
    h  = x + o(a);    n2 = RMSNorm(h);        y = h + down(SiLU(gate(n2)) * up(n2))

Two modes: a decode batch (one new token for each of B sequences, keys and values of `context` earlier tokens in a
cache) and a prefill (one sequence of T tokens, causal attention).  The linears go through `linears`, an object
with `one(name, x)` and `many(names, x)`: `LibraryLinears` calls the CUDA library (modules that share their input
as one group call), tests put a CPU reference in its place, and `FixedLinears` returns preallocated tensors so
that the rest of the layer can be timed alone.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import torch

HIDDEN, N_HEADS, N_KV_HEADS, HEAD_DIM, MLP = 4096, 32, 8, 128, 14336
ROPE_THETA = 500000.0
LINEARS = {"q": (HIDDEN, N_HEADS * HEAD_DIM), "k": (HIDDEN, N_KV_HEADS * HEAD_DIM), "v": (HIDDEN, N_KV_HEADS * HEAD_DIM),
           "o": (N_HEADS * HEAD_DIM, HIDDEN), "gate": (HIDDEN, MLP), "up": (HIDDEN, MLP), "down": (MLP, HIDDEN)}
GROUPS = (("q", "k", "v"), ("o",), ("gate", "up"), ("down",))


def rms_norm(x: torch.Tensor, g: torch.Tensor, eps: float = 1e-5) -> torch.Tensor:
    xf = x.float()
    return (xf * torch.rsqrt(xf.pow(2).mean(dim=-1, keepdim=True) + eps) * g.float()).to(x.dtype)


def rotary(t: torch.Tensor, positions: torch.Tensor) -> torch.Tensor:
    """Rotate-half rotary embedding; t[..., tokens, heads, HEAD_DIM], positions[tokens]."""
    half = HEAD_DIM // 2
    inv = ROPE_THETA ** (-torch.arange(0, half, device=t.device, dtype=torch.float32) / half)
    ang = positions.float()[:, None] * inv[None, :]
    cos, sin = ang.cos()[:, None, :], ang.sin()[:, None, :]
    tf = t.float()
    a, b = tf[..., :half], tf[..., half:]
    return torch.cat([a * cos - b * sin, b * cos + a * sin], dim=-1).to(t.dtype)


class LibraryLinears:
    """The seven MeteoRA linears through the CUDA library; modules that share x go out as one group call."""

    def __init__(self, weights: Dict[str, Dict[str, torch.Tensor]], k: int, grouped: bool = True):
        from . import binding
        self.mb, self.w, self.k, self.grouped = binding, weights, k, grouped
        self.ws: Dict[str, torch.Tensor] = {}
        self.routing: Dict[str, torch.Tensor] = {}

    def one(self, name: str, x: torch.Tensor) -> torch.Tensor:
        m = self.w[name]
        y, idx, _ = self.mb.meteora_linear_forward(x, m["W0"], m["A"], m["B"], m["Wg"], self.k,
                                                   workspace=self._workspace(name, x, [name]), return_routing=True)
        self.routing[name] = idx
        return y

    def many(self, names: Sequence[str], x: torch.Tensor) -> List[torch.Tensor]:
        if not self.grouped:
            return [self.one(n, x) for n in names]
        ms = [self.w[n] for n in names]
        ys, routing = self.mb.meteora_linear_forward_group(x, [m["W0"] for m in ms], [m["A"] for m in ms],
                                                           [m["B"] for m in ms], [m["Wg"] for m in ms], self.k,
                                                           workspace=self._workspace("+".join(names), x, names),
                                                           return_routing=True)
        for n, (idx, _) in zip(names, routing):
            self.routing[n] = idx
        return ys

    def _workspace(self, key: str, x: torch.Tensor, names: Sequence[str]) -> torch.Tensor:
        """One scratch buffer per call site, allocated on first use (so that a CUDA graph can be captured afterwards)."""
        key = f"{key}/{x.shape[0]}"
        if key not in self.ws:
            import ctypes
            lib, mb = self.mb.load_library(), self.mb
            N, r, _ = self.w[names[0]]["A"].shape
            d_outs = [int(self.w[n]["W0"].shape[0]) for n in names]
            shape = mb.make_shape(x.shape[0], x.shape[1], d_outs[0], N, r, self.k, x.dtype)
            n = (lib.meteora_group_workspace_bytes(ctypes.byref(shape), (ctypes.c_int * len(names))(*d_outs), len(names))
                 if len(names) > 1 else mb.meteora_workspace_bytes(shape))
            self.ws[key] = torch.zeros(n, dtype=torch.uint8, device=x.device)
        return self.ws[key]

    def status(self) -> int:
        return min([self.mb.meteora_workspace_status(ws) for ws in self.ws.values()] or [0])


class FixedLinears:
    """Stands in for the linears when the rest of the layer is timed alone: returns tensors made beforehand."""

    def __init__(self, T: int, dtype, device):
        g = torch.Generator(device=device).manual_seed(5)
        self.out = {n: torch.randn(T, d_out, device=device, generator=g).to(dtype) for n, (_, d_out) in LINEARS.items()}

    def one(self, name, x):
        return self.out[name]

    def many(self, names, x):
        return [self.out[n] for n in names]


def layer_forward(x: torch.Tensor, norms: Dict[str, torch.Tensor], linears, positions: torch.Tensor,
                  cache_k: Optional[torch.Tensor] = None, cache_v: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x[T, HIDDEN].  With a cache ([B, N_KV_HEADS, context, HEAD_DIM], B = T): decode, token t is the next token of
    sequence t at position positions[t].  Without: prefill of one sequence, causal attention over the T tokens."""
    T = x.shape[0]
    n1 = rms_norm(x, norms["input"])
    q, k, v = linears.many(("q", "k", "v"), n1)
    q = rotary(q.view(T, N_HEADS, HEAD_DIM), positions)
    k = rotary(k.view(T, N_KV_HEADS, HEAD_DIM), positions)
    v = v.view(T, N_KV_HEADS, HEAD_DIM)
    if cache_k is not None:
        keys = torch.cat([cache_k, k[:, :, None, :]], dim=2)                  # [B, 8, context + 1, 128]
        vals = torch.cat([cache_v, v[:, :, None, :]], dim=2)
        a = torch.nn.functional.scaled_dot_product_attention(q[:, :, None, :], keys, vals, enable_gqa=True)
        a = a.reshape(T, N_HEADS * HEAD_DIM)
    else:
        a = torch.nn.functional.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                                             v.transpose(0, 1)[None], is_causal=True, enable_gqa=True)
        a = a[0].transpose(0, 1).reshape(T, N_HEADS * HEAD_DIM)
    h = x + linears.one("o", a.contiguous())
    n2 = rms_norm(h, norms["post_attention"])
    gate, up = linears.many(("gate", "up"), n2)
    return h + linears.one("down", (torch.nn.functional.silu(gate.float()) * up.float()).to(x.dtype))


def random_layer(device, dtype=torch.bfloat16, N: int = 28, r: int = 8, seed: int = 11, b_std: float = 0.01):
    """Random weights of the layer's shapes, drawn on the device (distributions of the synthetic workloads)."""
    g = torch.Generator(device=device).manual_seed(seed)
    weights = {}
    for name, (d_in, d_out) in LINEARS.items():
        weights[name] = {"W0": (0.02 * torch.randn(d_out, d_in, device=device, generator=g)).to(dtype),
                         "A": ((torch.rand(N, r, d_in, device=device, generator=g) * 2 - 1) / math.sqrt(d_in)).to(dtype),
                         "B": (b_std * torch.randn(N, d_out, r, device=device, generator=g)).to(dtype),
                         "Wg": (torch.randn(N, d_in, device=device, generator=g) / math.sqrt(d_in)).to(dtype)}
    norms = {"input": (1.0 + 0.1 * torch.randn(HIDDEN, device=device, generator=g)).to(dtype),
             "post_attention": (1.0 + 0.1 * torch.randn(HIDDEN, device=device, generator=g)).to(dtype)}
    return weights, norms
